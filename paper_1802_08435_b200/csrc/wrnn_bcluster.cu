// Cluster-partitioned multi-row kernel (dense bf16 models, 2 or more rows advancing in lock step: the folded
// sub-tensors of Section 4 and the batched form of Section 2's sampling step).
//
// The rows of a batch are independent streams, so the batch is cut into groups of up to 64 rows and each group
// is given to one thread-block cluster of 16 CTAs.  Nothing ever crosses a cluster: the nine phases of a step
// (Fig. 1, Eq. 2) are separated by hardware cluster barriers instead of grid-wide ones, and clusters drift
// freely against one another.  Inside a cluster the weight rows are dealt out in chunks of eight rows:
//
//   A    a = R h_{t-1}                 CTA c holds the (u, r, e) rows of hidden-unit chunks c, c+16, c+32, ...
//   Gc   coarse gates -> y_c           from the TMEM accumulator of A
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
// the N side.  R is streamed every step from L2 (it is shared by all clusters) by TMA with the 128-byte swizzle,
// together with the activation tiles, through an mbarrier ring; the CTA's slices of O1 .. O4 stay resident in shared
// memory and the activations of those phases arrive in two multi-tile TMA copies.  Operands live in global memory
// as arrays of [rows][64] k-block tiles so that every copy is one box.  Accumulators live in TMEM (A: columns
// 0-255, kept until Gf; O1 / O3: 256-287; O2 / O4: 320-335).  The fp32 hidden state of a (row, unit) pair never
// leaves the registers of the thread that owns it; only its bf16 high / low split is written out (to L2, in the
// operand layout) for the next contractions.  Every mbarrier wait is bounded; a CTA whose wait ran out records it,
// skips its remaining tensor work and keeps arriving at the cluster barriers so that the launch drains cleanly.
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>

#include "wrnn_cluster.cuh"
#include "wrnn_internal.h"
#include "wrnn_tc.cuh"

namespace wrnn {

constexpr int BC_CS = 16;             // CTAs per cluster
constexpr int BC_THREADS = 512;
constexpr int BC_MAX_STAGES = 8;
constexpr int BC_SLACK = 16384;       // the 128-row A operand may read this far past a short activation tile
constexpr int BC_MROWS = 128;         // rows of an activation tile (the stacked operand of one cluster)
constexpr int BC_GROUP = 64;          // most rows of a batch one cluster takes
constexpr int BC_COL_A = 0, BC_COL_O1 = 256, BC_COL_O2 = 320, BC_TMEM_COLS = 512;
constexpr int BC_UH = 32;             // most hidden units of one half (coarse or fine) a CTA owns
constexpr int BC_S_BYTES = 3 * BC_UH * BC_GROUP * 4;       // staged accumulators [gate][unit][row] fp32
constexpr int BC_SOUT_PITCH = 40;                          // bf16 per (row, part) of the staged gate outputs
constexpr int BC_SOUT_BYTES = BC_GROUP * 2 * BC_SOUT_PITCH * 2;

struct BcPack {
    int H = 0, NCH = 0, NRp = 0, NOC = 0, NO1 = 0;
    __nv_bfloat16 *Wr = nullptr, *O1p = nullptr, *O2p = nullptr, *O3p = nullptr, *O4p = nullptr;   // [16][k-block][rows per CTA][64]
    float4 *Ip = nullptr;                                   // [16][3][64]: I of the CTA's gate rows
    float *bp = nullptr;                                    // [16][2][48]: b1 | b2 (head 0), b3 | b4 (head 1) of the CTA's rows
    __nv_bfloat16 *act[2] = {nullptr, nullptr};             // [clusters][H/64][128][64]   stacked high / low state tiles
    __nv_bfloat16 *q = nullptr;                             // [clusters][H/128][128][64]  stacked hidden-layer tiles
    CUtensorMap tmWr, tmO1, tmO2, tmO3, tmO4;
    int max_clusters = 0, max_dyn_smem = 0;
    int64_t weight_bytes = 0;
};

struct BcParams {
    int H, Hh, G, batch, RB, MR, NCH, NRp, NO1, n_stages, stage_bytes, kpart, res_bytes, s_off;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    int row_lag;                 // > 0: row b of the call is row_lag steps behind row b - 1 and takes one conditioning frame per step
    long long out_pitch;         // samples between the rows of `out`
    const float4 *Ip;
    const float *bp, *g;
    __nv_bfloat16 *act0, *act1, *q;
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;             // bound of every mbarrier wait
    int skip_cta; long long skip_step;       // self-test: this CTA's weight producer withholds its first load of this step (-1: none)
    alignas(64) CUtensorMap tmWr;
    alignas(64) CUtensorMap tmO1;
    alignas(64) CUtensorMap tmO2;
    alignas(64) CUtensorMap tmO3;
    alignas(64) CUtensorMap tmO4;
    alignas(64) CUtensorMap tmActA[2];     // one tile of MR rows (ring of phase A)
    alignas(64) CUtensorMap tmActO[2];     // kpart tiles of MR rows (operand of O1 / O3)
    alignas(64) CUtensorMap tmQ;           // kpart tiles of MR rows (operand of O2 / O4)
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

// element (operand row mrow, column k) of a cluster's tile array with nkb k-blocks
__device__ __forceinline__ size_t tile_index(int cl, int nkb, int mrow, int k)
{
    return (((size_t)cl * nkb + (k >> 6)) * BC_MROWS + mrow) * 64 + (k & 63);
}

#ifdef WRNN_PROFILE_BC
__device__ long long g_bcprof[32];
#define CSTAMP(i) do { if (threadIdx.x == 96) { const long long n_ = clock64(); s_prof[i] += n_ - bt_; bt_ = n_; } } while (0)
#define RBEGIN() long long rt_ = clock64()
#define RSTAMP(i) do { const long long n_ = clock64(); s_prof[i] += n_ - rt_; rt_ = n_; } while (0)
#else
#define CSTAMP(i) do { } while (0)
#define RBEGIN() do { } while (0)
#define RSTAMP(i) do { } while (0)
#endif

// DBG = false: plain sampling (no forced symbols, no dumps: what wrnn_sample runs)
template <bool DBG>
__global__ void __launch_bounds__(BC_THREADS, 1) bcluster_step_kernel(const __grid_constant__ BcParams p)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_full[BC_MAX_STAGES], s_empty[BC_MAX_STAGES], s_ofull[2], s_done, s_wload;
    __shared__ uint32_t s_tmem;
    __shared__ int s_failed;
    __shared__ float4 s_I[3 * 64];                  // [gate][unit of this CTA] -> (I0, I1, I2, -)
    __shared__ float s_b[2 * 48];                   // [head][b1 of the CTA's 32 hidden-layer rows | b2 of its 16 logits]
    __shared__ __align__(16) float s_log[4 * 256];  // logits of the rows this CTA draws for (row crank + 16 w of the group), written by peers
    __shared__ int s_c[BC_GROUP], s_f[BC_GROUP];    // c_t / f_t of every row of the group, broadcast by the drawing CTAs
#ifdef WRNN_PROFILE_BC
    __shared__ long long s_prof[32];
    long long bt_ = clock64();
    if (threadIdx.x < 32) s_prof[threadIdx.x] = 0;
#endif

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned crank;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    const int cl = blockIdx.x / BC_CS;
    const int row0 = cl * p.RB;
    const int nrows = min(p.RB, p.batch - row0);
    if (nrows <= 0) return;                         // the same for every CTA of the cluster
    const int H = p.H, Hh = p.Hh, NCH = p.NCH;
    const int nkbA = H / TC_BK, nkbH = Hh / TC_BK;

    // ---- fixed roles of this thread
    // (1) TMEM reader: warp (quadrant qd, slot); lanes 0-15 see the high-part rows 16 qd + lr, lanes 16-31 the low-part ones
    const int qd = warp & 3, slot = warp >> 2, half = lane >> 4, lr = lane & 15;
    const int nQ = (nrows + 15) >> 4;               // lane quadrants in use
    const int bl = 16 * qd + lr;
    const bool rowv = bl < nrows;
    const int gb = row0 + bl;
    const int mrow_hi = 32 * qd + lr, mrow_lo = mrow_hi + 16;
    // chunks of this CTA: i = 0 .. nchv-1 valid, the first nCc of them coarse
    const int tot_ch = H / 8, half_ch = Hh / 8;
    const int nchv = (tot_ch - (int)crank + BC_CS - 1) / BC_CS;
    const int nCc = (half_ch - (int)crank + BC_CS - 1) / BC_CS;
    // hidden-layer chunk (8 outputs of O1 / O3) of this warp
    const int och = (int)crank + BC_CS * slot;
    const bool ochv = och < half_ch;
    // (2) gate thread: one row of the group, hidden units g_u0, g_u0 + g_step, ... of the half in flight
    const int rshift = nrows <= 16 ? 4 : (nrows <= 32 ? 5 : 6);
    const int g_row = tid & ((1 << rshift) - 1), g_u0 = tid >> rshift, g_step = BC_THREADS >> rshift;
    const bool g_rowv = g_row < nrows;
    const int g_gb = row0 + g_row;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t res0 = smem_u32(base);                           // resident O1 | O3 | O2 | O4 tiles
    const uint32_t wO1 = res0, wO3 = wO1 + (uint32_t)(nkbH * p.NO1 * 128), wO2 = wO3 + (uint32_t)(nkbH * p.NO1 * 128),
                   wO4 = wO2 + (uint32_t)(nkbH * 16 * 128);
    uint8_t *area = base + p.res_bytes;
    const uint32_t area0 = smem_u32(area);                          // ring of phase A / operand of the O phases
    float *S = reinterpret_cast<float *>(area + p.s_off);           // staged accumulators [gate][unit][row]
    __nv_bfloat16 *Sout = reinterpret_cast<__nv_bfloat16 *>(area + p.s_off + BC_S_BYTES);
    const uint32_t done_bar = smem_u32(&s_done);
    volatile int *failed = &s_failed;
    const uint32_t abytes = (uint32_t)p.MR * 128u;

    if (tid == 0) {
        for (int i = 0; i < BC_MAX_STAGES; ++i) { mbar_init(smem_u32(&s_full[i]), 2); mbar_init(smem_u32(&s_empty[i]), 1); }
        mbar_init(smem_u32(&s_ofull[0]), 1); mbar_init(smem_u32(&s_ofull[1]), 1);
        mbar_init(done_bar, 1);
        mbar_init(smem_u32(&s_wload), 1);
        s_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // resident slices of O1 .. O4: one box each
        const uint32_t wb = smem_u32(&s_wload);
        mbar_expect_tx(wb, (uint32_t)p.res_bytes);
        tma_load_2d(wO1, &p.tmO1, wb, 0, (int)crank * nkbH * p.NO1);
        tma_load_2d(wO3, &p.tmO3, wb, 0, (int)crank * nkbH * p.NO1);
        tma_load_2d(wO2, &p.tmO2, wb, 0, (int)crank * nkbH * 16);
        tma_load_2d(wO4, &p.tmO4, wb, 0, (int)crank * nkbH * 16);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(BC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (int i = tid; i < 3 * 64; i += BC_THREADS) s_I[i] = p.Ip[(size_t)crank * 3 * 64 + i];
    for (int i = tid; i < 2 * 48; i += BC_THREADS) s_b[i] = p.bp[(size_t)crank * 96 + i];
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    auto fail = [&](int step, int phase) {
        *failed = 1;
        if (atomicCAS(&p.status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) { p.status->cta = blockIdx.x; p.status->step = step; p.status->phase = phase; }
    };
    if (!mbar_wait(smem_u32(&s_wload), 0, p.limit_ns)) fail(-1, 0);

    // ---- initial state: fp32 in the registers of the gate threads, stacked high / low tiles in buffer 0
    // (operand rows that no thread writes were zeroed by the host)
    float hc[4], hf[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int uc = g_u0 + j * g_step;
        hc[j] = hf[j] = 0.f;
        if (g_rowv && p.h_in) {
            if (uc < 8 * nCc) hc[j] = p.h_in[(size_t)g_gb * H + 8 * ((int)crank + BC_CS * (uc >> 3)) + (uc & 7)];
            if (uc < 8 * (nchv - nCc)) hf[j] = p.h_in[(size_t)g_gb * H + 8 * ((int)crank + BC_CS * (nCc + (uc >> 3))) + (uc & 7)];
        }
        if (g_rowv) {
            const int mr_hi = 32 * (g_row >> 4) + (g_row & 15);
            if (uc < 8 * nCc) {
                const int unit = 8 * ((int)crank + BC_CS * (uc >> 3)) + (uc & 7);
                const __nv_bfloat16 hi = __float2bfloat16_rn(hc[j]);
                p.act0[tile_index(cl, nkbA, mr_hi, unit)] = hi;
                p.act0[tile_index(cl, nkbA, mr_hi + 16, unit)] = __float2bfloat16_rn(hc[j] - __bfloat162float(hi));
            }
            if (uc < 8 * (nchv - nCc)) {
                const int unit = 8 * ((int)crank + BC_CS * (nCc + (uc >> 3))) + (uc & 7);
                const __nv_bfloat16 hi = __float2bfloat16_rn(hf[j]);
                p.act0[tile_index(cl, nkbA, mr_hi, unit)] = hi;
                p.act0[tile_index(cl, nkbA, mr_hi + 16, unit)] = __float2bfloat16_rn(hf[j] - __bfloat162float(hi));
            }
        }
    }
    // the rows this CTA draws for: row crank + 16 w by warp w; their last drawn (or forced) pair stays in registers
    const int s_r = (int)crank + BC_CS * warp;
    const bool sampler = warp < 4 && s_r < nrows;
    const int s_gb = row0 + s_r;
    // The three single-thread roles of the contractions sit on lane 31 of warps 1, 3 and 5: as gate threads those lanes serve
    // the last row slot of the group, which is empty unless the group has exactly 16, 32 or 64 rows, so that their role work
    // does not delay gate work of their own.
    const int role = (lane == 31 && (warp == 1 || warp == 3 || warp == 5)) ? (warp >> 1) : -1;   // 0: MMA issue, 1 / 2: TMA producers
    int last_c = sampler ? (p.c_in ? (int)p.c_in[s_gb] : 128) : 0, last_f = sampler ? (p.f_in ? (int)p.f_in[s_gb] : 0) : 0;
    fence_proxy_async();
    cluster_barrier();

    // ring position of the three role threads of phase A (they walk the same sequence of k-blocks), parities of the
    // O-phase operand barriers and of `done`
    int rst = 0;
    uint32_t rph = 0, oph = 0, dph = 0;

    // Only the MMA thread watches the `done` mbarrier; everybody else blocks on the CTA barrier, so that no polling warp
    // competes with the three role threads for issue slots.
    auto wait_done = [&](int step, int phase) {
        if (warp == 1) {
            if (role == 0) {
                RBEGIN();
                if (!*failed && !mbar_wait(done_bar, dph, p.limit_ns)) fail(step, phase);
                RSTAMP(31);
            }
            __syncwarp();
        }
        dph ^= 1;
        __syncthreads();
        tc_fence_after();
    };

    // Phase A: D[128 x NRp] (TMEM column 0) = state tiles of buffer `cur` . (this CTA's rows of R)^T through the ring.
    // One role thread loads the activation tiles, one the weight tiles, one issues the MMAs.
    // The role loops are kept to a handful of instructions per k-block: a lone thread issues slowly.
    const uint32_t full0 = smem_u32(&s_full[0]), empty0 = smem_u32(&s_empty[0]);
    auto gemm_a_issue = [&](int cur, int step) {
        if (role >= 0 && !*failed) {
            if (role == 0) {
                const uint32_t idesc = umma_idesc_bf16(128, p.NRp);
                const uint32_t dstep = (uint32_t)(p.stage_bytes >> 4), boff = abytes >> 4;
                uint32_t da = umma_desc_lo(area0) + (uint32_t)rst * dstep;
                bool ok = true;
                RBEGIN();
                for (int kb = 0; kb < nkbA; ++kb) {
                    if (!mbar_wait(full0 + 8u * (uint32_t)rst, rph, p.limit_ns)) { ok = false; break; }
                    tc_fence_after();
                    umma_bf16_kblock(tmem + BC_COL_A, da, da + boff, idesc, kb ? 1u : 0u);
                    umma_commit(empty0 + 8u * (uint32_t)rst);
                    da += dstep;
                    if (++rst == p.n_stages) { rst = 0; rph ^= 1; da = umma_desc_lo(area0); }
                }
                if (ok) umma_commit(done_bar);
                else fail(step, 1);
            } else {
                const bool is_act = role == 1;
                const uint32_t bytes = is_act ? abytes : (uint32_t)p.NRp * 128u;
                const CUtensorMap *tmA = &p.tmActA[cur];
                uint32_t dst = area0 + (uint32_t)rst * (uint32_t)p.stage_bytes + (is_act ? 0u : abytes);
                int coord = is_act ? cl * nkbA : (int)crank * nkbA * p.NRp;
                const int cstep = is_act ? 1 : p.NRp;
                RBEGIN();
                // (the writers of the state tiles and of this shared memory issued their proxy fences before the cluster barrier)
                for (int kb = 0; kb < nkbA; ++kb) {
                    if (!mbar_wait(empty0 + 8u * (uint32_t)rst, rph ^ 1, p.limit_ns)) { fail(step, 1); break; }
                    const uint32_t fb = full0 + 8u * (uint32_t)rst;
                    mbar_expect_tx(fb, bytes);
                    if (is_act) tma_load_3d(dst, tmA, fb, 0, 0, coord);
                    else if (!(kb == 0 && (int)blockIdx.x == p.skip_cta && step == p.skip_step)) tma_load_2d(dst, &p.tmWr, fb, 0, coord);
                    coord += cstep;
                    dst += (uint32_t)p.stage_bytes;
                    if (++rst == p.n_stages) { rst = 0; rph ^= 1; dst -= (uint32_t)p.n_stages * (uint32_t)p.stage_bytes; }
                }
            }
        }
    };

    // O phases: D[128 x n_w] (TMEM column dcol) = tiles tile0 .. tile0 + nkbH - 1 of an activation array . (resident weights)^T.
    // The operand arrives as two copies of kpart tiles; the MMAs of the first half start while the second is in flight.
    auto gemm_o_issue = [&](const CUtensorMap *tmA, int tile0, uint32_t wres, int n_w, uint32_t dcol, int step, int phase) {
        if (role >= 0 && !*failed) {
            if (role != 0) {
                // one producer fetches the first half of the operand, the other the second
                const int part = role - 1;
                const uint32_t half_bytes = (uint32_t)p.kpart * abytes, fb = smem_u32(&s_ofull[part]);
                mbar_expect_tx(fb, half_bytes);
                tma_load_3d(area0 + (uint32_t)part * half_bytes, tmA, fb, 0, 0, tile0 + part * p.kpart);
            } else {
                const uint32_t idesc = umma_idesc_bf16(128, n_w);
                const uint32_t astep = abytes >> 4, wstep = (uint32_t)(n_w * 8);
                uint32_t da = umma_desc_lo(area0), db = umma_desc_lo(wres);
                RBEGIN();
                bool ok = mbar_wait(smem_u32(&s_ofull[0]), oph, p.limit_ns);
                RSTAMP(30);
                if (ok) {
                    tc_fence_after();
                    int kb = 0;
                    for (; kb < p.kpart; ++kb, da += astep, db += wstep) umma_bf16_kblock(tmem + dcol, da, db, idesc, kb ? 1u : 0u);
                    RSTAMP(27);
                    ok = mbar_wait(smem_u32(&s_ofull[1]), oph, p.limit_ns);
                    RSTAMP(28);
                    if (ok) {
                        tc_fence_after();
                        for (; kb < nkbH; ++kb, da += astep, db += wstep) umma_bf16_kblock(tmem + dcol, da, db, idesc, 1u);
                    }
                    RSTAMP(29);
                }
                if (ok) umma_commit(done_bar);
                else fail(step, phase);
            }
        }
        oph ^= 1;
    };

    // Inputs of the gates of one half that do not depend on the contraction (I x + conditioning; x2 joins later for the
    // fine half): computed while the tensor pipe works.
    auto gate_inputs = [&](bool coarse, float x0, float x1, const float *grow, float (&pre)[4][3]) {
        const int i0 = coarse ? 0 : nCc, nchh = coarse ? nCc : nchv - nCc;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int uh = g_u0 + j * g_step;
            pre[j][0] = pre[j][1] = pre[j][2] = 0.f;
            if (!g_rowv || uh >= 8 * nchh) continue;
            const int il = 8 * (i0 + (uh >> 3)) + (uh & 7);
            const int unit = 8 * ((int)crank + BC_CS * (i0 + (uh >> 3))) + (uh & 7);
            const float4 Iu = s_I[il], Ir = s_I[64 + il], Ie = s_I[128 + il];
            pre[j][0] = fmaf(Iu.x, x0, fmaf(Iu.y, x1, __ldg(grow + unit)));
            pre[j][1] = fmaf(Ir.x, x0, fmaf(Ir.y, x1, __ldg(grow + H + unit)));
            pre[j][2] = fmaf(Ie.x, x0, fmaf(Ie.y, x1, __ldg(grow + 2 * H + unit)));
        }
    };

    // Gates of Eq. 2 for the hidden units of one half that this CTA owns (coarse: x2 = 0; fine: x2 = c_t).
    auto gates = [&](bool coarse, long long s, float x2, const float (&pre)[4][3], __nv_bfloat16 *anext, float (&hreg)[4]) {
        const int i0 = coarse ? 0 : nCc, nchh = coarse ? nCc : nchv - nCc;      // chunk slots of this half
        // (1) accumulator columns of the half: TMEM -> shared memory, high-part + low-part products added on the way;
        // the warp of slot g takes gate g: its 8 nchh (<= 32) columns are adjacent
        if (qd < nQ && slot < 3) {
            float v[32];
            tmem_ld32(tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_A + 8 * NCH * slot + 8 * i0, v);
            tmem_wait_ld();
            float *d = S + ((size_t)(slot * BC_UH)) * BC_GROUP + bl;
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                // lanes 0-15 (high-part products) keep the even column, lanes 16-31 (low-part) the odd one
                const float mine = half ? v[c + 1] : v[c], send = half ? v[c] : v[c + 1];
                const float sum = mine + __shfl_xor_sync(0xffffffffu, send, 16);
                if (c < 8 * nchh) d[(size_t)(c + half) * BC_GROUP] = sum;
            }
        }
        CSTAMP(22);
        __syncthreads();
        CSTAMP(23);
        // (2) one (row, unit) pair per thread and pass
        if (g_rowv) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int uh = g_u0 + j * g_step;
                if (uh >= 8 * nchh) continue;
                const int il = 8 * (i0 + (uh >> 3)) + (uh & 7);               // unit of this CTA
                const float au = S[(size_t)uh * BC_GROUP + g_row], ar = S[(size_t)(BC_UH + uh) * BC_GROUP + g_row],
                            ae = S[(size_t)(2 * BC_UH + uh) * BC_GROUP + g_row];
                float pu = pre[j][0], pr = pre[j][1], pe = pre[j][2];
                if (!coarse) { pu = fmaf(s_I[il].z, x2, pu); pr = fmaf(s_I[64 + il].z, x2, pr); pe = fmaf(s_I[128 + il].z, x2, pe); }
                const float u = sigmoidf_fast(au + pu), r = sigmoidf_fast(ar + pr);
                const float e = tanhf_fast(fmaf(r, ae, pe));
                const float hn = fmaf(u, hreg[j], (1.0f - u) * e);
                hreg[j] = hn;
                const __nv_bfloat16 hi = __float2bfloat16_rn(hn);
                Sout[(size_t)(2 * g_row) * BC_SOUT_PITCH + uh] = hi;
                Sout[(size_t)(2 * g_row + 1) * BC_SOUT_PITCH + uh] = __float2bfloat16_rn(hn - __bfloat162float(hi));
                if (DBG && (p.dbg_gates || p.dbg_h)) {
                    const int unit = 8 * ((int)crank + BC_CS * (i0 + (uh >> 3))) + (uh & 7);
                    if (p.dbg_gates) { float *d = p.dbg_gates + ((size_t)s * p.batch + g_gb) * p.G + unit; d[0] = u; d[H] = r; d[2 * H] = e; }
                    if (p.dbg_h) p.dbg_h[((size_t)s * p.batch + g_gb) * H + unit] = hn;
                }
            }
        }
        CSTAMP(24);
        __syncthreads();
        CSTAMP(25);
        // (3) 16-byte pieces (row, part, chunk) into the next state tiles
        {
            const int ii = tid & 3, part = (tid >> 2) & 1, row = tid >> 3;
            if (ii < nchh && row < nrows) {
                const uint4 v = *reinterpret_cast<const uint4 *>(Sout + (size_t)(2 * row + part) * BC_SOUT_PITCH + 8 * ii);
                const int mrow = 32 * (row >> 4) + 16 * part + (row & 15);
                *reinterpret_cast<uint4 *>(anext + tile_index(cl, nkbA, mrow, 8 * ((int)crank + BC_CS * (i0 + ii)))) = v;
            }
        }
    };

    // conditioning frame of this thread's row, tracked without a division per step
    long long g_frame = 0;
    int g_rem = 0;
    float x0 = 0.f, x1 = 0.f;
    if (g_rowv) {
        const long long pos = p.row_lag > 0 ? 0 : p.step0 * p.row_stride + (long long)(p.stream0 + (unsigned)g_gb) * p.row_offset_mul;
        g_frame = pos / p.hop;
        g_rem = (int)(pos - g_frame * p.hop);
        x0 = scale8(p.c_in ? (int)p.c_in[g_gb] : 128);
        x1 = scale8(p.f_in ? (int)p.f_in[g_gb] : 0);
    }

    for (long long s = 0; s < p.n_steps; ++s) {
        __nv_bfloat16 *anext = (s & 1) ? p.act0 : p.act1;
        const int cur = (int)(s & 1);
        const float *grow = p.g + ((size_t)g_gb * p.n_frames + (size_t)g_frame) * p.G;
        float pre[4][3];
        // ---- A + Gc
        CSTAMP(0);
        gemm_a_issue(cur, (int)s);
        if (s > 0 && g_rowv) x1 = scale8(s_f[g_row]);                  // f_{t-1}: drawn at the end of the last step
        gate_inputs(true, x0, x1, grow, pre);
        wait_done((int)s, 1);
        CSTAMP(1);
        gates(true, s, 0.f, pre, anext, hc);
        CSTAMP(26);
        fence_proxy_async();
        CSTAMP(2);
        cluster_barrier();
        CSTAMP(3);
        float x2 = 0.f;

        for (int head = 0; head < 2; ++head) {
            const float *bh = s_b + 48 * head;
            // ---- O1 / O3: hidden layer on this half of the new state
            gemm_o_issue(&p.tmActO[cur ^ 1], cl * nkbA + head * nkbH, head ? wO3 : wO1, p.NO1, BC_COL_O1, (int)s, 2 + 4 * head);
            if (head == 0) gate_inputs(false, x0, x1, grow, pre);            // for Gf, while the tensor pipe works
            wait_done((int)s, 2 + 4 * head);
            CSTAMP(4 + 8 * head);
            if (qd < nQ && 8 * slot < p.NO1) {
                float v[8];
                tmem_ld8(tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_O1 + 8 * slot, v);
                tmem_wait_ld();
                __nv_bfloat16 o[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float t = v[e] + __shfl_xor_sync(0xffffffffu, v[e], 16);
                    const float x = fmaxf(t + bh[8 * slot + e], 0.f);
                    // both half-warps hold the sums: the lower writes the high parts, the upper the low parts
                    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                    o[e] = half ? __float2bfloat16_rn(x - __bfloat162float(hi)) : hi;
                }
                if (rowv && ochv) *reinterpret_cast<uint4 *>(p.q + tile_index(cl, nkbH, half ? mrow_lo : mrow_hi, 8 * och)) = pack8_bf16(o);
            }
            fence_proxy_async();
            CSTAMP(5 + 8 * head);
            cluster_barrier();
            CSTAMP(6 + 8 * head);
            // ---- O2 / O4: logits 16 crank .. + 15
            gemm_o_issue(&p.tmQ, cl * nkbH, head ? wO4 : wO2, 16, BC_COL_O2, (int)s, 3 + 4 * head);
            wait_done((int)s, 3 + 4 * head);
            CSTAMP(7 + 8 * head);
            if (qd < nQ && slot < 2) {
                float v[8];
                tmem_ld8(tmem + ((uint32_t)(32 * qd) << 16) + BC_COL_O2 + 8 * slot, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] += __shfl_xor_sync(0xffffffffu, v[e], 16);
                if (rowv) {
                    const int c0 = 8 * slot + 4 * half;                        // four logits per lane
                    float4 o;
                    o.x = (half ? v[4] : v[0]) + bh[32 + c0 + 0];
                    o.y = (half ? v[5] : v[1]) + bh[32 + c0 + 1];
                    o.z = (half ? v[6] : v[2]) + bh[32 + c0 + 2];
                    o.w = (half ? v[7] : v[3]) + bh[32 + c0 + 3];
                    const int r0 = 16 * (int)crank + c0;
                    // row bl of the group is drawn by warp bl / 16 of CTA bl % 16: the logits go straight into its shared memory
                    const unsigned dst = map_to_rank(smem_addr(s_log + (bl >> 4) * 256 + r0), (unsigned)(bl & 15));
                    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(o.x), "f"(o.y), "f"(o.z), "f"(o.w) : "memory");
                    if (DBG && p.dbg_logits) *reinterpret_cast<float4 *>(p.dbg_logits + (((size_t)s * p.batch + gb) * 2 + head) * 256 + r0) = o;
                }
            }
            CSTAMP(8 + 8 * head);
            cluster_barrier();
            CSTAMP(9 + 8 * head);
            // ---- Sc / Sf: softmax + inverse-CDF draw, one warp per row; the result goes to every CTA of the cluster
            int drawn = 0, used = 0;
            const size_t s_o = (size_t)s_gb * p.n_steps + s;
            if (sampler) {
                float l[8];
                const float4 v0 = *reinterpret_cast<const float4 *>(s_log + warp * 256 + 8 * lane);
                const float4 v1 = *reinterpret_cast<const float4 *>(s_log + warp * 256 + 8 * lane + 4);
                l[0] = v0.x; l[1] = v0.y; l[2] = v0.z; l[3] = v0.w; l[4] = v1.x; l[5] = v1.y; l[6] = v1.z; l[7] = v1.w;
                const float u = uniform24(p.seed, p.stream0 + (unsigned)s_gb, (unsigned long long)(p.step0 + s - (long long)s_gb * p.row_lag), head);
                drawn = warp_softmax_draw_scan(l, u, lane);
                const uint8_t *forced = head ? p.f_forced : p.c_forced;
                used = (DBG && forced) ? (int)forced[s_o] : drawn;
                if (lane < BC_CS) {
                    const unsigned dst = map_to_rank(smem_addr((head ? s_f : s_c) + s_r), (unsigned)lane);
                    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(dst), "r"(used) : "memory");
                }
            }
            CSTAMP(10 + 8 * head);
            cluster_barrier();
            CSTAMP(11 + 8 * head);
            // outputs leave after the barrier so that its release does not wait for them
            if (sampler) {
                if (head == 0) {
                    if (lane == 0 && p.c_out) p.c_out[s_o] = (uint8_t)drawn;
                    last_c = used;
                } else {
                    if (lane == 0) {
                        if (p.f_out) p.f_out[s_o] = (uint8_t)drawn;
                        if (p.out) p.out[(long long)s_gb * p.out_pitch + s] = (int16_t)(256 * last_c + used - 32768);
                    }
                    last_f = used;
                }
            }
            if (head == 0) {
                // ---- Gf: fine gates, now that c_t is known (it reaches only these rows, Section 2)
                x2 = g_rowv ? scale8(s_c[g_row]) : 0.f;
                gates(false, s, x2, pre, anext, hf);
                CSTAMP(26);
                fence_proxy_async();
                CSTAMP(20);
                cluster_barrier();
                CSTAMP(21);
            }
        }
        x0 = x2;                                  // c_t becomes c_{t-1}
        g_rem += p.row_stride;
        while (g_rem >= p.hop) { g_rem -= p.hop; ++g_frame; }
    }

    if (p.h_out && g_rowv) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int uc = g_u0 + j * g_step;
            if (uc < 8 * nCc) p.h_out[(size_t)g_gb * H + 8 * ((int)crank + BC_CS * (uc >> 3)) + (uc & 7)] = hc[j];
            if (uc < 8 * (nchv - nCc)) p.h_out[(size_t)g_gb * H + 8 * ((int)crank + BC_CS * (nCc + (uc >> 3))) + (uc & 7)] = hf[j];
        }
    }
    if (sampler && lane == 0) {
        if (p.c_st_out) p.c_st_out[s_gb] = (uint8_t)last_c;
        if (p.f_st_out) p.f_st_out[s_gb] = (uint8_t)last_f;
    }
#ifdef WRNN_PROFILE_BC
    if (blockIdx.x == 0 && tid == 96) for (int i = 0; i < 32; ++i) g_bcprof[i] += s_prof[i];
#endif
    tc_fence_before();
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(BC_TMEM_COLS) : "memory");
}

// ---------------------------------------------------------------------------------------------
static int round_up(int x, int m) { return (x + m - 1) / m * m; }

// Rows of a dense matrix (bf16 bits, `cols` wide) dealt out in chunks of 8 rows -- CTA c gets chunks c, c + 16, ... of
// each of the `gates` row blocks of `rows_per_gate` rows, as row 8 nch g + 8 i + e of its slice, padded with zero
// rows to rp rows -- and cut into 64-column k-block tiles: [c][k-block][rp][64].
static std::vector<uint16_t> deal_rows(const std::vector<uint16_t> &dense, int cols, int gates, int rows_per_gate, int nch, int rp)
{
    const int nkb = cols / 64;
    std::vector<uint16_t> out((size_t)BC_CS * nkb * rp * 64, 0);
    for (int c = 0; c < BC_CS; ++c)
        for (int g = 0; g < gates; ++g)
            for (int i = 0; i < nch; ++i) {
                const int ch = c + BC_CS * i;
                if (ch >= rows_per_gate / 8) continue;
                for (int e = 0; e < 8; ++e)
                    for (int kb = 0; kb < nkb; ++kb)
                        std::memcpy(&out[(((size_t)c * nkb + kb) * rp + (size_t)g * 8 * nch + 8 * i + e) * 64],
                                    &dense[((size_t)g * rows_per_gate + 8 * ch + e) * cols + 64 * kb], 128);
            }
    return out;
}

// rows 16 c .. 16 c + 15 of a dense [256][cols] matrix as [c][k-block][16][64]
static std::vector<uint16_t> tile_logit_rows(const std::vector<uint16_t> &dense, int cols)
{
    const int nkb = cols / 64;
    std::vector<uint16_t> out((size_t)256 * cols, 0);
    for (int c = 0; c < BC_CS; ++c)
        for (int kb = 0; kb < nkb; ++kb)
            for (int r = 0; r < 16; ++r)
                std::memcpy(&out[(((size_t)c * nkb + kb) * 16 + r) * 64], &dense[((size_t)16 * c + r) * cols + 64 * kb], 128);
    return out;
}

struct BcGeometry { int n_cl, RB, MR, stage_bytes, n_stages, kpart, res_bytes, s_off, smem; bool fits; };

static BcGeometry bc_geometry(const BcPack &k, int batch)
{
    BcGeometry g;
    int ncl = (batch + 15) / 16;
    if (ncl > k.max_clusters) ncl = k.max_clusters;
    g.RB = (batch + ncl - 1) / ncl;
    g.n_cl = (batch + g.RB - 1) / g.RB;
    g.MR = 32 * ((g.RB + 15) / 16);
    const int nkbH = k.H / 128;
    g.kpart = (nkbH + 1) / 2;
    g.res_bytes = 2 * nkbH * 128 * (k.NO1 + 16);
    g.stage_bytes = (g.MR + k.NRp) * 128;
    g.s_off = round_up(2 * g.kpart * g.MR * 128, 1024);
    const int area = k.max_dyn_smem - 1024 - g.res_bytes;
    int ns = (area - BC_SLACK) / g.stage_bytes;
    if (ns > BC_MAX_STAGES) ns = BC_MAX_STAGES;
    g.n_stages = ns;
    int need = ns * g.stage_bytes + BC_SLACK;
    const int need_o = g.s_off + BC_S_BYTES + BC_SOUT_BYTES;
    if (need_o > need) need = need_o;
    g.fits = ns >= 2 && need_o <= area && g.RB <= BC_GROUP;
    g.smem = 1024 + g.res_bytes + need;
    return g;
}

int bcluster_supported(const wrnn_model *m, int batch, std::string *why)
{
    if (!m->bcluster) { if (why) *why = "model was not packed for the cluster-partitioned kernel"; return WRNN_ERR_UNSUPPORTED; }
    if (batch < 2) { if (why) *why = "cluster-partitioned kernel needs at least two rows"; return WRNN_ERR_UNSUPPORTED; }
    if (!bc_geometry(*m->bcluster, batch).fits) { if (why) *why = "batch does not fit the co-resident clusters"; return WRNN_ERR_UNSUPPORTED; }
    return WRNN_OK;
}

int bcluster_prepare(wrnn_model *m)
{
    if (m->dtype != WRNN_BF16 || m->sparse) { m->err = "cluster-partitioned kernel takes dense bf16 models"; return WRNN_ERR_UNSUPPORTED; }
    if (m->H % 128 != 0 || m->H > 1024) { m->err = "cluster-partitioned kernel needs H to be a multiple of 128, at most 1024"; return WRNN_ERR_UNSUPPORTED; }
    if (m->max_batch < 2) { m->err = "max_batch < 2"; return WRNN_ERR_UNSUPPORTED; }
    if (!encode_tiled_fn()) { m->err = "driver has no tensor-map encoder"; return WRNN_ERR_UNSUPPORTED; }
    BcPack *k = new BcPack();
    m->bcluster = k;
    const int H = m->H, Hh = H / 2, nkbA = H / 64, nkbH = Hh / 64;
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
    if (cudaFuncGetAttributes(&fa, bcluster_step_kernel<true>) != cudaSuccess) return failed("cluster-partitioned kernel image missing", WRNN_ERR_CUDA);
    k->max_dyn_smem = dev_smem - (int)fa.sharedSizeBytes;
    if (cudaFuncSetAttribute(bcluster_step_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, k->max_dyn_smem) != cudaSuccess ||
        cudaFuncSetAttribute(bcluster_step_kernel<true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(bcluster_step_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, k->max_dyn_smem) != cudaSuccess ||
        cudaFuncSetAttribute(bcluster_step_kernel<false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        return failed("cluster-partitioned kernel attributes rejected", WRNN_ERR_UNSUPPORTED);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(BC_CS); cfg.blockDim = dim3(BC_THREADS); cfg.dynamicSmemBytes = (size_t)k->max_dyn_smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = BC_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, bcluster_step_kernel<true>, &cfg) != cudaSuccess || n < 1)
            return failed("device cannot co-schedule a 16-CTA cluster of this size", WRNN_ERR_UNSUPPORTED);
        k->max_clusters = n;
    }
    if (!bc_geometry(*k, m->max_batch).fits) return failed("max_batch does not fit the co-resident clusters", WRNN_ERR_UNSUPPORTED);

    auto up = [&](const std::vector<uint16_t> &v, __nv_bfloat16 **dst) {
        k->weight_bytes += (int64_t)v.size() * 2;
        return cudaMalloc((void **)dst, v.size() * 2) == cudaSuccess && cudaMemcpy(*dst, v.data(), v.size() * 2, cudaMemcpyHostToDevice) == cudaSuccess;
    };
    bool ok = up(deal_rows(dense_bf16_bits(m->hR), H, 3, H, k->NCH, k->NRp), &k->Wr) &&
              up(deal_rows(dense_bf16_bits(m->hO1), Hh, 1, Hh, k->NOC, k->NO1), &k->O1p) &&
              up(deal_rows(dense_bf16_bits(m->hO3), Hh, 1, Hh, k->NOC, k->NO1), &k->O3p) &&
              up(tile_logit_rows(dense_bf16_bits(m->hO2), Hh), &k->O2p) && up(tile_logit_rows(dense_bf16_bits(m->hO4), Hh), &k->O4p);
    {
        std::vector<float4> Ih((size_t)BC_CS * 3 * 64, make_float4(0.f, 0.f, 0.f, 0.f));
        std::vector<float> bh((size_t)BC_CS * 96, 0.f);
        for (int c = 0; c < BC_CS; ++c) {
            for (int g = 0; g < 3; ++g)
                for (int i = 0; i < k->NCH; ++i) {
                    const int ch = c + BC_CS * i;
                    if (ch >= H / 8) continue;
                    for (int e = 0; e < 8; ++e) {
                        const float *src = &m->hI[(size_t)(g * H + 8 * ch + e) * 3];
                        Ih[((size_t)c * 3 + g) * 64 + 8 * i + e] = make_float4(src[0], src[1], src[2], 0.f);
                    }
                }
            for (int head = 0; head < 2; ++head) {
                const std::vector<float> &ba = head ? m->hb3 : m->hb1, &bb = head ? m->hb4 : m->hb2;
                for (int i = 0; i < k->NOC; ++i) {
                    const int ch = c + BC_CS * i;
                    if (ch >= Hh / 8) continue;
                    for (int e = 0; e < 8; ++e) bh[(size_t)c * 96 + 48 * head + 8 * i + e] = ba.empty() ? 0.f : ba[8 * ch + e];
                }
                for (int r = 0; r < 16; ++r) bh[(size_t)c * 96 + 48 * head + 32 + r] = bb.empty() ? 0.f : bb[16 * c + r];
            }
        }
        ok = ok && cudaMalloc((void **)&k->Ip, Ih.size() * sizeof(float4)) == cudaSuccess &&
             cudaMemcpy(k->Ip, Ih.data(), Ih.size() * sizeof(float4), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMalloc((void **)&k->bp, bh.size() * 4) == cudaSuccess &&
             cudaMemcpy(k->bp, bh.data(), bh.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
    }
    const size_t tile = (size_t)BC_MROWS * 64 * 2, ncl = (size_t)k->max_clusters;
    ok = ok && cudaMalloc((void **)&k->act[0], ncl * nkbA * tile) == cudaSuccess && cudaMalloc((void **)&k->act[1], ncl * nkbA * tile) == cudaSuccess &&
         cudaMalloc((void **)&k->q, ncl * nkbH * tile) == cudaSuccess;
    ok = ok && make_map(&k->tmWr, k->Wr, (long long)BC_CS * nkbA * k->NRp, 64, k->NRp) &&
         make_map(&k->tmO1, k->O1p, (long long)BC_CS * nkbH * k->NO1, 64, nkbH * k->NO1) &&
         make_map(&k->tmO3, k->O3p, (long long)BC_CS * nkbH * k->NO1, 64, nkbH * k->NO1) &&
         make_map(&k->tmO2, k->O2p, (long long)BC_CS * nkbH * 16, 64, nkbH * 16) &&
         make_map(&k->tmO4, k->O4p, (long long)BC_CS * nkbH * 16, 64, nkbH * 16);
    if (!ok) return failed("device allocation for the cluster-partitioned kernel failed", WRNN_ERR_NOMEM);
    return WRNN_OK;
}

void bcluster_destroy(wrnn_model *m)
{
    BcPack *k = m->bcluster;
    if (!k) return;
    cudaFree(k->Wr); cudaFree(k->O1p); cudaFree(k->O2p); cudaFree(k->O3p); cudaFree(k->O4p); cudaFree(k->Ip); cudaFree(k->bp);
    cudaFree(k->act[0]); cudaFree(k->act[1]); cudaFree(k->q);
    delete k;
    m->bcluster = nullptr;
}

int bcluster_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes)
{
    const BcPack &k = *m->bcluster;
    const BcGeometry g = bc_geometry(k, batch);
    if (n_ctas) *n_ctas = g.n_cl * BC_CS;
    if (n_threads) *n_threads = BC_THREADS;
    if (smem) *smem = g.smem;
    if (weight_bytes) *weight_bytes = k.weight_bytes;
    return WRNN_OK;
}

int bcluster_run(wrnn_model *m, const StepArgs &a, cudaStream_t s)
{
    BcPack &k = *m->bcluster;
    const BcGeometry g = bc_geometry(k, a.batch);
    BcParams p;
    std::memset(&p, 0, sizeof(p));
    p.RB = g.RB; p.MR = g.MR; p.stage_bytes = g.stage_bytes; p.n_stages = g.n_stages; p.kpart = g.kpart; p.res_bytes = g.res_bytes; p.s_off = g.s_off;
    p.H = m->H; p.Hh = m->H / 2; p.G = 3 * m->H; p.batch = a.batch;
    p.NCH = k.NCH; p.NRp = k.NRp; p.NO1 = k.NO1;
    p.n_steps = a.n_steps; p.step0 = a.step0; p.stream0 = a.stream0; p.seed = a.seed;
    p.n_frames = m->cond_dim ? a.n_frames : 1;
    p.hop = m->cond_dim ? a.hop : 1;
    p.row_stride = m->cond_dim ? a.row_stride : 0;
    p.row_offset_mul = m->cond_dim ? a.row_offset_mul : 0;
    p.Ip = k.Ip; p.bp = k.bp; p.g = m->g;
    p.act0 = k.act[0]; p.act1 = k.act[1]; p.q = k.q;
    p.h_in = a.h_in; p.h_out = a.h_out; p.c_in = a.c_in; p.f_in = a.f_in; p.c_st_out = a.c_st_out; p.f_st_out = a.f_st_out;
    p.c_forced = a.c_forced; p.f_forced = a.f_forced; p.c_out = a.c_out; p.f_out = a.f_out; p.out = a.out;
    p.row_lag = a.row_lag; p.out_pitch = a.out_pitch ? a.out_pitch : a.n_steps;
    p.dbg_gates = a.dbg_gates; p.dbg_h = a.dbg_h; p.dbg_logits = a.dbg_logits;
    p.status = m->status;
    p.limit_ns = m->wait_limit_ns(); p.skip_cta = m->dbg_skip_cta; p.skip_step = m->dbg_skip_step;
    p.tmWr = k.tmWr; p.tmO1 = k.tmO1; p.tmO2 = k.tmO2; p.tmO3 = k.tmO3; p.tmO4 = k.tmO4;
    const int nkbA = m->H / 64, nkbH = m->H / 128;
    const long long tilesA = (long long)k.max_clusters * nkbA, tilesH = (long long)k.max_clusters * nkbH;
    bool ok = make_map_tiles(&p.tmQ, k.q, tilesH, BC_MROWS, g.MR, g.kpart);
    for (int b = 0; b < 2; ++b)
        ok = ok && make_map_tiles(&p.tmActA[b], k.act[b], tilesA, BC_MROWS, g.MR, 1) && make_map_tiles(&p.tmActO[b], k.act[b], tilesA, BC_MROWS, g.MR, g.kpart);
    if (!ok) { m->err = "tensor-map encoding failed"; return WRNN_ERR_CUDA; }
    // operand rows that no thread writes must read as zero
    const size_t tile = (size_t)BC_MROWS * 64 * 2;
    if (cudaMemsetAsync(k.act[0], 0, (size_t)tilesA * tile, s) != cudaSuccess || cudaMemsetAsync(k.act[1], 0, (size_t)tilesA * tile, s) != cudaSuccess ||
        cudaMemsetAsync(k.q, 0, (size_t)tilesH * tile, s) != cudaSuccess || cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess)
        return WRNN_ERR_CUDA;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.n_cl * BC_CS); cfg.blockDim = dim3(BC_THREADS); cfg.dynamicSmemBytes = (size_t)g.smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = BC_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const bool teacher = p.c_forced || p.f_forced || p.dbg_gates || p.dbg_h || p.dbg_logits;
    const cudaError_t e = teacher ? cudaLaunchKernelEx(&cfg, bcluster_step_kernel<true>, p) : cudaLaunchKernelEx(&cfg, bcluster_step_kernel<false>, p);
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
