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
// that arrival of the data is the signal.  Inside a cluster the hidden layer and the logits travel
// through distributed shared memory the same way.  The fine head of step t overlaps the recurrent
// product of step t+1 (f_t is only needed by the coarse gates of t+1).
//
// Every wait is bounded; a CTA that gives up records where, raises the abort word and all CTAs
// leave through the final cluster barrier.
#include <cooperative_groups.h>

#include <algorithm>
#include <cstring>

#include "wrnn_internal.h"

namespace cg = cooperative_groups;

namespace wrnn {

struct ResidentPack {
    int NC = 0, CS = 0, NCTA = 0, UC = 0, HR = 0, LR = 0, K = 0, KC = 0, NW = 0;
    int n_rrows = 0;                 // 6 UC
    size_t blob_bytes = 0;           // per CTA: bf16 weights then fp32 small parameters
    size_t w_bytes = 0;              // bf16 part of the blob
    uint8_t *d_blob = nullptr;       // [NCTA][blob_bytes]
    unsigned long long *d_slots = nullptr;   // [2 halves][2 parities][K] (value, tag)
    int smem_bytes = 0;
    int64_t weight_bytes_per_step = 0;
};

struct ResidentParams {
    int H, K, KC, UC, HR, LR, CS, n_rrows;
    long long n_steps, step0;
    unsigned stream0;
    unsigned long long seed;
    int n_frames, hop, row_stride, row_offset_mul;
    const uint8_t *blob; unsigned long long blob_bytes, w_bytes;
    const float *g;                          // [n_frames][3H]
    unsigned long long *slots;               // [2][2][K]
    const float *h_in; float *h_out;
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;
    uint8_t *c_out, *f_out;
    int16_t *out;
    float *dbg_gates, *dbg_h, *dbg_logits;
    DevStatus *status;
    unsigned long long limit_ns;
};

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned map_to_rank(unsigned addr, unsigned rank)
{
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// 16-byte store into a (possibly remote) CTA's shared memory: two (value, tag) pairs.
__device__ __forceinline__ void st_cluster_ll(unsigned addr, float v0, float v1, unsigned tag)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(__float_as_uint(v0)), "r"(tag),
                 "r"(__float_as_uint(v1)), "r"(tag)
                 : "memory");
}
__device__ __forceinline__ uint4 ld_shared_volatile_v4(unsigned addr)
{
    uint4 v;
    asm volatile("ld.volatile.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Bounded-wait bookkeeping shared by all polls of a thread.
struct Waiter {
    DevStatus *status;
    unsigned long long limit_ns;

    // called every few thousand failed polls; true = give up (somebody else already did, or time ran out)
    __device__ __forceinline__ bool expired(unsigned long long &t0, int step, int phase)
    {
        if (ld_relaxed_s32(&status->code) != DEV_OK) return true;
        const unsigned long long now = globaltimer_ns();
        if (t0 == 0) { t0 = now; return false; }
        if (now - t0 > limit_ns) {
            if (atomicCAS(&status->code, DEV_OK, DEV_TIMEOUT) == DEV_OK) {
                status->cta = blockIdx.x; status->step = step; status->phase = phase;
            }
            return true;
        }
        return false;
    }
};

// Lane's share of an input vector of KC 8-float chunks: chunks lane, lane + 32, ...
template <int CPL>
__device__ __forceinline__ void load_vec(const float *vec, int KC, int lane, float (&hv)[CPL * 8])
{
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const int ch = lane + 32 * i;
        if (ch < KC) {
            const float4 a = *reinterpret_cast<const float4 *>(vec + 8 * ch);
            const float4 b = *reinterpret_cast<const float4 *>(vec + 8 * ch + 4);
            hv[8 * i] = a.x; hv[8 * i + 1] = a.y; hv[8 * i + 2] = a.z; hv[8 * i + 3] = a.w;
            hv[8 * i + 4] = b.x; hv[8 * i + 5] = b.y; hv[8 * i + 6] = b.z; hv[8 * i + 7] = b.w;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) hv[8 * i + k] = 0.f;
        }
    }
}

// Four consecutive bf16 rows (KC 16-byte chunks each, contiguous in shared memory) times the
// lane's vector share; returns with lane l holding the total of row (l & 3).
template <int CPL>
__device__ __forceinline__ float dot4(const uint4 *w, int KC, int lane, const float (&hv)[CPL * 8])
{
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const int ch = lane + 32 * i;
        if (ch < KC) {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint4 v = w[r * KC + ch];
                float s = acc[r];
                s = fmaf(bf16lo(v.x), hv[8 * i], s);     s = fmaf(bf16hi(v.x), hv[8 * i + 1], s);
                s = fmaf(bf16lo(v.y), hv[8 * i + 2], s); s = fmaf(bf16hi(v.y), hv[8 * i + 3], s);
                s = fmaf(bf16lo(v.z), hv[8 * i + 4], s); s = fmaf(bf16hi(v.z), hv[8 * i + 5], s);
                s = fmaf(bf16lo(v.w), hv[8 * i + 6], s); s = fmaf(bf16hi(v.w), hv[8 * i + 7], s);
                acc[r] = s;
            }
        }
    }
    return warp_reduce_scatter<4>(acc, lane);
}

template <int CPL>
__global__ void __launch_bounds__(768, 1) resident_dense_kernel(const ResidentParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cta = blockIdx.x;                       // global CTA index = owner index of state units
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, KC = p.KC, UC = p.UC, HR = p.HR, LR = p.LR, CS = p.CS, H = p.H;
    const int NR = p.n_rrows;                          // 6 UC

    // ---- shared memory carve-up (must match resident_smem_bytes)
    const uint4 *wRA = reinterpret_cast<const uint4 *>(smem);                 // [NR][KC]  R rows x coarse columns
    const uint4 *wRB = wRA + (size_t)NR * KC;                                  // [NR][KC]  R rows x fine columns
    const uint4 *wO1 = wRB + (size_t)NR * KC;                                  // [HR][KC]
    const uint4 *wO3 = wO1 + (size_t)HR * KC;
    const uint4 *wO2 = wO3 + (size_t)HR * KC;                                  // [LR][KC]
    const uint4 *wO4 = wO2 + (size_t)LR * KC;
    const float *sI = reinterpret_cast<const float *>(smem + p.w_bytes);       // [NR][3]
    const float *sb1 = sI + NR * 3, *sb3 = sb1 + HR, *sb2 = sb3 + HR, *sb4 = sb2 + LR;
    float *vecC = reinterpret_cast<float *>(smem + p.blob_bytes);              // [K] y_c
    float *vecF = vecC + K;                                                    // [K] y_f
    float *qvec = vecF + K;                                                    // [K] hidden layer of the head
    float *a_part = qvec + K;                                                  // [NR] R[:, :Hh] y_c
    float *a_full = a_part + NR;                                               // [NR] R h
    uint4 *qbuf = reinterpret_cast<uint4 *>(a_full + NR + ((2 * NR) % 4 ? 4 - (2 * NR) % 4 : 0));   // [2][K/2]
    uint4 *lbuf = qbuf + K;                                                    // [2][128]

    // ---- one-time load of this CTA's weights
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.blob + (size_t)cta * p.blob_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>(smem);
        for (size_t i = tid; i < p.blob_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        for (int i = tid; i < K + 256; i += blockDim.x) qbuf[i] = make_uint4(0, 0, 0, 0);   // qbuf and lbuf are adjacent
        for (int i = tid; i < K; i += blockDim.x) {
            vecC[i] = p.h_in ? p.h_in[i] : 0.f;
            vecF[i] = p.h_in ? p.h_in[K + i] : 0.f;
        }
    }
    __syncthreads();
    cluster.sync();     // peers' exchange buffers are zeroed before anyone writes into them

    Waiter wt{p.status, p.limit_ns};
    bool my_bad = false;      // this thread gave up on a wait; made CTA-uniform by __syncthreads_or
    const int n_head_warps = HR / 4, n_r_warps = NR / 4, n_logit_warps = LR / 4;
    const bool is_head_warp = warp < n_head_warps;
    const bool is_r_warp = warp >= n_head_warps && warp < n_head_warps + n_r_warps;
    const int r_task = warp - n_head_warps;
    const bool writer = (cta == 0);

    // warp 0 keeps the stream's scalar state
    int c_prev = p.c_in ? p.c_in[0] : 128, f_prev = p.f_in ? p.f_in[0] : 0;
    float hC = 0.f, hF = 0.f;
    if (warp == 0 && lane < UC) { hC = vecC[cta * UC + lane]; hF = vecF[cta * UC + lane]; }

    // prologue: a_part = R[:, :Hh] y_c(-1)
    if (is_r_warp) {
        float hv[CPL * 8];
        load_vec<CPL>(vecC, KC, lane, hv);
        const float t = dot4<CPL>(wRA + (size_t)(4 * r_task) * KC, KC, lane, hv);
        if (lane < 4) a_part[4 * r_task + lane] = t;
    }
    __syncthreads();

    unsigned hs = 0;            // cluster-exchange counter (one per head evaluation)
    const long long T = p.n_steps;

    for (long long s = 0; s <= T; ++s) {
        // conditioning rows of this CTA's units, fetched early (they do not depend on the chain)
        float gC[3] = {0.f, 0.f, 0.f}, gF[3] = {0.f, 0.f, 0.f};
        int cf_next = -1, ff_prev = -1;
        if (warp == 0) {
            if (lane < UC && s < T) {
                const long long fr = ((p.step0 + s) * p.row_stride + (long long)p.stream0 * p.row_offset_mul) / p.hop;
                const float *g = p.g + (size_t)fr * 3 * H;
#pragma unroll
                for (int gate = 0; gate < 3; ++gate) {
                    gC[gate] = __ldg(g + gate * H + cta * UC + lane);
                    gF[gate] = __ldg(g + gate * H + K + cta * UC + lane);
                }
            }
            if (p.c_forced && s < T) cf_next = p.c_forced[s];
            if (p.f_forced && s > 0) ff_prev = p.f_forced[s - 1];
        }

        // =================== fine half: head of step s-1 (draw f_{s-1}) + R[:, Hh:] y_f(s-1)
        if (s > 0) {
            const unsigned long long *slots = p.slots + (size_t)(2 + ((s - 1) & 1)) * K;
            const unsigned tag = (unsigned)s;                 // y_f(s-1) carries tag s
            for (int i = tid; i < K; i += blockDim.x) {
                unsigned long long v, t0 = 0; unsigned n = 0;
                while ((unsigned)((v = ld_relaxed_u64(slots + i)) >> 32) != tag)
                    if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 1)) { my_bad = true; break; }
                vecF[i] = __uint_as_float((unsigned)v);
            }
            if (__syncthreads_or(my_bad)) break;
        }
        if (is_head_warp && s > 0) {
            float hv[CPL * 8];
            load_vec<CPL>(vecF, KC, lane, hv);
            const int r0 = 4 * warp;
            const float t = dot4<CPL>(wO3 + (size_t)r0 * KC, KC, lane, hv);
            const float q0 = fmaxf(__shfl_sync(FULL, t, 0) + sb3[r0], 0.f), q1 = fmaxf(__shfl_sync(FULL, t, 1) + sb3[r0 + 1], 0.f);
            const float q2 = fmaxf(__shfl_sync(FULL, t, 2) + sb3[r0 + 2], 0.f), q3 = fmaxf(__shfl_sync(FULL, t, 3) + sb3[r0 + 3], 0.f);
            if (lane < 2 * CS) {
                const int peer = lane >> 1, pair = lane & 1;
                const unsigned a = map_to_rank(smem_addr(qbuf + (size_t)(hs & 1) * (K / 2) + (rank * HR + r0) / 2 + pair), peer);
                st_cluster_ll(a, pair ? q2 : q0, pair ? q3 : q1, hs + 1);
            }
        } else if (is_r_warp) {
            float hv[CPL * 8];
            load_vec<CPL>(vecF, KC, lane, hv);
            const float t = dot4<CPL>(wRB + (size_t)(4 * r_task) * KC, KC, lane, hv);
            if (lane < 4) a_full[4 * r_task + lane] = a_part[4 * r_task + lane] + t;
        }
        if (s > 0) {
            for (int i = tid; i < K / 2; i += blockDim.x) {
                const unsigned a = smem_addr(qbuf + (size_t)(hs & 1) * (K / 2) + i);
                uint4 v; unsigned long long t0 = 0; unsigned n = 0;
                while (true) {
                    v = ld_shared_volatile_v4(a);
                    if (v.y == hs + 1 && v.w == hs + 1) break;
                    if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 2)) { my_bad = true; break; }
                }
                qvec[2 * i] = __uint_as_float(v.x); qvec[2 * i + 1] = __uint_as_float(v.z);
            }
        }
        if (__syncthreads_or(my_bad)) break;
        if (s > 0 && warp < n_logit_warps) {
            float hv[CPL * 8];
            load_vec<CPL>(qvec, KC, lane, hv);
            const int r0 = 4 * warp;
            const float t = dot4<CPL>(wO4 + (size_t)r0 * KC, KC, lane, hv);
            const float l0 = __shfl_sync(FULL, t, 0) + sb4[r0], l1 = __shfl_sync(FULL, t, 1) + sb4[r0 + 1];
            const float l2 = __shfl_sync(FULL, t, 2) + sb4[r0 + 2], l3 = __shfl_sync(FULL, t, 3) + sb4[r0 + 3];
            if (lane < 2 * CS) {
                const int peer = lane >> 1, pair = lane & 1;
                const unsigned a = map_to_rank(smem_addr(lbuf + (size_t)(hs & 1) * 128 + (rank * LR + r0) / 2 + pair), peer);
                st_cluster_ll(a, pair ? l2 : l0, pair ? l3 : l1, hs + 1);
            }
        }
        if (warp == 0) {
            if (s > 0) {
                float l[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const unsigned a = smem_addr(lbuf + (size_t)(hs & 1) * 128 + 4 * lane + k);
                    uint4 v; unsigned long long t0 = 0; unsigned n = 0;
                    while (true) {
                        v = ld_shared_volatile_v4(a);
                        if (v.y == hs + 1 && v.w == hs + 1) break;
                        if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 3)) { my_bad = true; break; }
                    }
                    l[2 * k] = __uint_as_float(v.x); l[2 * k + 1] = __uint_as_float(v.z);
                }
                my_bad = __any_sync(FULL, my_bad);
                const float u = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + s - 1), 1u);
                int f = warp_softmax_draw(l, u, lane);
                if (writer) {
                    if (p.dbg_logits) {
                        float *d = p.dbg_logits + ((size_t)(s - 1) * 2 + 1) * 256 + 8 * lane;
#pragma unroll
                        for (int k = 0; k < 8; ++k) d[k] = l[k];
                    }
                    if (lane == 0 && p.f_out) p.f_out[s - 1] = (uint8_t)f;
                }
                if (ff_prev >= 0) f = ff_prev;
                if (writer && lane == 0 && p.out) p.out[s - 1] = (int16_t)(256 * c_prev + f - 32768);
                f_prev = f;
            }
        }
        if (s > 0) ++hs;
        if (s == T) break;

        // coarse gates of step s (Eq. 2; c_t does not reach these rows)
        if (warp == 0 && lane < UC && !my_bad) {
            const float x0 = scale8(c_prev), x1 = scale8(f_prev);
            const float *Iu = sI + 3 * (0 * UC + lane), *Ir = sI + 3 * (1 * UC + lane), *Ie = sI + 3 * (2 * UC + lane);
            const float pu = a_full[lane] + fmaf(Iu[0], x0, fmaf(Iu[1], x1, gC[0]));
            const float pr = a_full[UC + lane] + fmaf(Ir[0], x0, fmaf(Ir[1], x1, gC[1]));
            const float pe = fmaf(Ie[0], x0, fmaf(Ie[1], x1, gC[2]));
            const float u = sigmoidf_acc(pu), r = sigmoidf_acc(pr);
            const float e = tanhf(fmaf(r, a_full[2 * UC + lane], pe));
            hC = fmaf(u, hC, (1.0f - u) * e);
            const int j = cta * UC + lane;
            st_relaxed_u64(p.slots + (size_t)(s & 1) * K + j, ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hC));
            if (p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[j] = u; d[H + j] = r; d[2 * H + j] = e; }
            if (p.dbg_h) p.dbg_h[(size_t)s * H + j] = hC;
        }

        // =================== coarse half: head of step s (draw c_s) + R[:, :Hh] y_c(s) for step s+1
        {
            const unsigned long long *slots = p.slots + (size_t)(s & 1) * K;
            const unsigned tag = (unsigned)(s + 1);
            for (int i = tid; i < K; i += blockDim.x) {
                unsigned long long v, t0 = 0; unsigned n = 0;
                while ((unsigned)((v = ld_relaxed_u64(slots + i)) >> 32) != tag)
                    if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 4)) { my_bad = true; break; }
                vecC[i] = __uint_as_float((unsigned)v);
            }
            if (__syncthreads_or(my_bad)) break;
        }
        if (is_head_warp) {
            float hv[CPL * 8];
            load_vec<CPL>(vecC, KC, lane, hv);
            const int r0 = 4 * warp;
            const float t = dot4<CPL>(wO1 + (size_t)r0 * KC, KC, lane, hv);
            const float q0 = fmaxf(__shfl_sync(FULL, t, 0) + sb1[r0], 0.f), q1 = fmaxf(__shfl_sync(FULL, t, 1) + sb1[r0 + 1], 0.f);
            const float q2 = fmaxf(__shfl_sync(FULL, t, 2) + sb1[r0 + 2], 0.f), q3 = fmaxf(__shfl_sync(FULL, t, 3) + sb1[r0 + 3], 0.f);
            if (lane < 2 * CS) {
                const int peer = lane >> 1, pair = lane & 1;
                const unsigned a = map_to_rank(smem_addr(qbuf + (size_t)(hs & 1) * (K / 2) + (rank * HR + r0) / 2 + pair), peer);
                st_cluster_ll(a, pair ? q2 : q0, pair ? q3 : q1, hs + 1);
            }
        } else if (is_r_warp) {
            float hv[CPL * 8];
            load_vec<CPL>(vecC, KC, lane, hv);
            const float t = dot4<CPL>(wRA + (size_t)(4 * r_task) * KC, KC, lane, hv);
            if (lane < 4) a_part[4 * r_task + lane] = t;
        }
        for (int i = tid; i < K / 2; i += blockDim.x) {
            const unsigned a = smem_addr(qbuf + (size_t)(hs & 1) * (K / 2) + i);
            uint4 v; unsigned long long t0 = 0; unsigned n = 0;
            while (true) {
                v = ld_shared_volatile_v4(a);
                if (v.y == hs + 1 && v.w == hs + 1) break;
                if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 5)) { my_bad = true; break; }
            }
            qvec[2 * i] = __uint_as_float(v.x); qvec[2 * i + 1] = __uint_as_float(v.z);
        }
        if (__syncthreads_or(my_bad)) break;
        if (warp < n_logit_warps) {
            float hv[CPL * 8];
            load_vec<CPL>(qvec, KC, lane, hv);
            const int r0 = 4 * warp;
            const float t = dot4<CPL>(wO2 + (size_t)r0 * KC, KC, lane, hv);
            const float l0 = __shfl_sync(FULL, t, 0) + sb2[r0], l1 = __shfl_sync(FULL, t, 1) + sb2[r0 + 1];
            const float l2 = __shfl_sync(FULL, t, 2) + sb2[r0 + 2], l3 = __shfl_sync(FULL, t, 3) + sb2[r0 + 3];
            if (lane < 2 * CS) {
                const int peer = lane >> 1, pair = lane & 1;
                const unsigned a = map_to_rank(smem_addr(lbuf + (size_t)(hs & 1) * 128 + (rank * LR + r0) / 2 + pair), peer);
                st_cluster_ll(a, pair ? l2 : l0, pair ? l3 : l1, hs + 1);
            }
        }
        if (warp == 0) {
            float l[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned a = smem_addr(lbuf + (size_t)(hs & 1) * 128 + 4 * lane + k);
                uint4 v; unsigned long long t0 = 0; unsigned n = 0;
                while (true) {
                    v = ld_shared_volatile_v4(a);
                    if (v.y == hs + 1 && v.w == hs + 1) break;
                    if ((++n & 4095u) == 0 && wt.expired(t0, (int)s, 6)) { my_bad = true; break; }
                }
                l[2 * k] = __uint_as_float(v.x); l[2 * k + 1] = __uint_as_float(v.z);
            }
            my_bad = __any_sync(FULL, my_bad);
            const float u = uniform24(p.seed, p.stream0, (unsigned long long)(p.step0 + s), 0u);
            int c = warp_softmax_draw(l, u, lane);
            if (writer) {
                if (p.dbg_logits) {
                    float *d = p.dbg_logits + ((size_t)s * 2) * 256 + 8 * lane;
#pragma unroll
                    for (int k = 0; k < 8; ++k) d[k] = l[k];
                }
                if (lane == 0 && p.c_out) p.c_out[s] = (uint8_t)c;
            }
            if (cf_next >= 0) c = cf_next;

            // fine gates of step s: now c_s is known (I* lets it reach only these rows)
            if (lane < UC && !my_bad) {
                const float x0 = scale8(c_prev), x1 = scale8(f_prev), x2 = scale8(c);
                const float *Iu = sI + 3 * (3 * UC + lane), *Ir = sI + 3 * (4 * UC + lane), *Ie = sI + 3 * (5 * UC + lane);
                const float pu = a_full[3 * UC + lane] + fmaf(Iu[0], x0, fmaf(Iu[1], x1, fmaf(Iu[2], x2, gF[0])));
                const float pr = a_full[4 * UC + lane] + fmaf(Ir[0], x0, fmaf(Ir[1], x1, fmaf(Ir[2], x2, gF[1])));
                const float pe = fmaf(Ie[0], x0, fmaf(Ie[1], x1, fmaf(Ie[2], x2, gF[2])));
                const float u2 = sigmoidf_acc(pu), r2 = sigmoidf_acc(pr);
                const float e2 = tanhf(fmaf(r2, a_full[5 * UC + lane], pe));
                hF = fmaf(u2, hF, (1.0f - u2) * e2);
                const int j = cta * UC + lane;
                st_relaxed_u64(p.slots + (size_t)(2 + (s & 1)) * K + j, ((unsigned long long)(unsigned)(s + 1) << 32) | __float_as_uint(hF));
                if (p.dbg_gates) { float *d = p.dbg_gates + (size_t)s * 3 * H; d[K + j] = u2; d[H + K + j] = r2; d[2 * H + K + j] = e2; }
                if (p.dbg_h) p.dbg_h[(size_t)s * H + K + j] = hF;
            }
            c_prev = c;
        }
        ++hs;
    }

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
static int resident_smem_bytes(const ResidentPack &k)
{
    size_t b = k.blob_bytes;
    b += (size_t)3 * k.K * 4;                       // vecC, vecF, qvec
    size_t a = (size_t)2 * k.n_rrows;               // a_part, a_full
    a += (a % 4) ? 4 - (a % 4) : 0;
    b += a * 4;
    b += (size_t)k.K * 16;                          // qbuf [2][K/2] x 16 B
    b += 256 * 16;                                  // lbuf [2][128] x 16 B
    return (int)b;
}

static uint16_t bf16_bits_of(float rounded)
{
    uint32_t b;
    std::memcpy(&b, &rounded, 4);
    return (uint16_t)(b >> 16);
}

// dense row `row` of a host block-row matrix -> bf16 bits for columns [c0, c0 + n)
static void dense_row_bf16(const BsrHost &M, int row, int c0, int n, uint16_t *dst)
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

static bool choose_shape(const wrnn_model *m, ResidentPack *k, std::string *why)
{
    const int H = m->H, Hh = H / 2;
    if (m->dtype != WRNN_BF16) { if (why) *why = "resident kernel stores bf16 weights only"; return false; }
    if (m->sparse) { if (why) *why = "resident dense kernel does not take block masks"; return false; }
    if (H % 16 != 0 || Hh / 8 > 64) { if (why) *why = "H must be a multiple of 16 and at most 1024"; return false; }
    const int CS = 8;
    if (Hh % (4 * CS) != 0) { if (why) *why = "H/2 must be a multiple of 32"; return false; }
    int best = 0;
    for (int ncta = CS; ncta <= m->n_sms; ncta += CS) {
        if (Hh % ncta) continue;
        const int uc = Hh / ncta;
        if (uc % 2 || uc > 32) continue;
        const int nw = Hh / CS / 4 + 6 * uc / 4;
        if (nw > 24 || nw < 8) continue;
        best = ncta;
    }
    if (!best) { if (why) *why = "no CTA count divides H/2 suitably"; return false; }
    k->CS = CS; k->NCTA = best; k->NC = best / CS; k->UC = Hh / best; k->HR = Hh / CS; k->LR = 256 / CS;
    k->K = Hh; k->KC = Hh / 8; k->n_rrows = 6 * k->UC;
    k->NW = k->HR / 4 + k->n_rrows / 4;
    k->w_bytes = ((size_t)2 * k->n_rrows + 2 * k->HR + 2 * k->LR) * k->K * 2;
    size_t small = ((size_t)k->n_rrows * 3 + 2 * k->HR + 2 * k->LR) * 4;
    small = (small + 15) / 16 * 16;
    k->blob_bytes = k->w_bytes + small;
    k->smem_bytes = resident_smem_bytes(*k);
    return true;
}

static void *resident_fn() { return (void *)resident_dense_kernel<2>; }

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
    ResidentPack k;
    std::string why;
    if (!choose_shape(m, &k, &why)) { m->err = why; return WRNN_ERR_UNSUPPORTED; }
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, m->device);
    if ((size_t)k.smem_bytes > prop.sharedMemPerBlockOptin) { m->err = "weights do not fit in shared memory"; return WRNN_ERR_UNSUPPORTED; }
    if (cudaFuncSetAttribute(resident_fn(), cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem_bytes) != cudaSuccess) {
        cudaGetLastError(); m->err = "cannot raise the dynamic shared memory limit"; return WRNN_ERR_UNSUPPORTED;
    }
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    fill_launch(k, &cfg, at, 0, false);
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, resident_fn(), &cfg) != cudaSuccess || max_clusters < k.NC) {
        cudaGetLastError(); m->err = "not enough co-resident clusters on this device"; return WRNN_ERR_UNSUPPORTED;
    }

    // ---- per-CTA blobs
    const int H = m->H, K = k.K, UC = k.UC;
    std::vector<uint8_t> blob((size_t)k.NCTA * k.blob_bytes, 0);
    std::vector<uint16_t> row(K);
    for (int cta = 0; cta < k.NCTA; ++cta) {
        const int rank = cta % k.CS;
        uint8_t *base = blob.data() + (size_t)cta * k.blob_bytes;
        uint16_t *w = reinterpret_cast<uint16_t *>(base);
        float *sm = reinterpret_cast<float *>(base + k.w_bytes);
        // R rows: index (half * 3 + gate) * UC + u  ->  matrix row gate * H + half * K + cta * UC + u
        for (int part = 0; part < 2; ++part)            // 0: coarse columns (RA), 1: fine columns (RB)
            for (int rr = 0; rr < k.n_rrows; ++rr) {
                const int half = rr / (3 * UC), gate = (rr / UC) % 3, u = rr % UC;
                const int mrow = gate * H + half * K + cta * UC + u;
                dense_row_bf16(m->hR, mrow, part * K, K, row.data());
                std::memcpy(w + ((size_t)part * k.n_rrows + rr) * K, row.data(), (size_t)K * 2);
                if (part == 0) for (int c = 0; c < 3; ++c) sm[rr * 3 + c] = m->hI[(size_t)mrow * 3 + c];
            }
        uint16_t *wo = w + (size_t)2 * k.n_rrows * K;
        const BsrHost *Oa[2] = {&m->hO1, &m->hO3}, *Ob[2] = {&m->hO2, &m->hO4};
        for (int h = 0; h < 2; ++h)
            for (int r = 0; r < k.HR; ++r) {
                dense_row_bf16(*Oa[h], rank * k.HR + r, 0, K, row.data());
                std::memcpy(wo + ((size_t)h * k.HR + r) * K, row.data(), (size_t)K * 2);
            }
        uint16_t *wl = wo + (size_t)2 * k.HR * K;
        for (int h = 0; h < 2; ++h)
            for (int r = 0; r < k.LR; ++r) {
                dense_row_bf16(*Ob[h], rank * k.LR + r, 0, K, row.data());
                std::memcpy(wl + ((size_t)h * k.LR + r) * K, row.data(), (size_t)K * 2);
            }
        float *b = sm + k.n_rrows * 3;
        for (int r = 0; r < k.HR; ++r) { b[r] = m->hb1[rank * k.HR + r]; b[k.HR + r] = m->hb3[rank * k.HR + r]; }
        b += 2 * k.HR;
        for (int r = 0; r < k.LR; ++r) { b[r] = m->hb2[rank * k.LR + r]; b[k.LR + r] = m->hb4[rank * k.LR + r]; }
    }
    ResidentPack *pk = new ResidentPack(k);
    bool ok = cudaMalloc((void **)&pk->d_blob, blob.size()) == cudaSuccess &&
              cudaMemcpy(pk->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMalloc((void **)&pk->d_slots, (size_t)4 * K * 8) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(pk->d_blob); cudaFree(pk->d_slots);
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
    p.H = m->H; p.K = k.K; p.KC = k.KC; p.UC = k.UC; p.HR = k.HR; p.LR = k.LR; p.CS = k.CS; p.n_rrows = k.n_rrows;
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
    p.status = m->status;
    p.limit_ns = 2000000000ull;

    if (cudaMemsetAsync(k.d_slots, 0, (size_t)4 * k.K * 8, s) != cudaSuccess) return WRNN_ERR_CUDA;
    if (cudaMemsetAsync(m->status, 0, sizeof(DevStatus), s) != cudaSuccess) return WRNN_ERR_CUDA;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[2];
    fill_launch(k, &cfg, at, s, true);
    cudaError_t e = cudaLaunchKernelEx(&cfg, resident_dense_kernel<2>, p);
    if (e != cudaSuccess) {
        m->err = std::string("resident kernel launch failed: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return WRNN_ERR_CUDA;
    }
    ++g_launches;
    return WRNN_OK;
}

}  // namespace wrnn
