// Device helpers shared by the cluster-resident single-stream kernels: distributed-shared-memory
// exchange primitives (tagged 16-byte stores, volatile polls), bounded waits, the exact 3-way bf16 split
// of an fp32 vector in MMA B-fragment order, and the straight-line m16n8k16 tile product.
#pragma once
#include <cuda_bf16.h>

#include "wrnn_device.cuh"

namespace wrnn {

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
// Asynchronous 16-byte (or, below, 8-byte) store of four (two) values into a (possibly remote) CTA's shared memory that counts its bytes on an
// mbarrier of the same CTA: the receiver waits on the barrier instead of polling the data, so nothing competes with the
// arriving stores (measured on a 16-CTA all-gather of 448 values: 600 cycles against 780 for tagged stores + polls).
__device__ __forceinline__ void st_async_v4(unsigned addr, float v0, float v1, float v2, float v3, unsigned mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
                 "r"(__float_as_uint(v0)), "r"(__float_as_uint(v1)), "r"(__float_as_uint(v2)), "r"(__float_as_uint(v3)), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v2(unsigned addr, float v0, float v1, unsigned mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];" ::"r"(addr),
                 "r"(__float_as_uint(v0)), "r"(__float_as_uint(v1)), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ void mbar_init_cluster(unsigned mbar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
// one arrival that also announces `bytes` of asynchronous stores still to come in this phase
__device__ __forceinline__ void mbar_arrive_expect(unsigned mbar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_parity(unsigned mbar, unsigned parity)
{
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }" : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    return ok != 0;
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
    __device__ __noinline__ bool expired(unsigned long long &t0, int step, int phase)
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

// Split image of an fp32 input vector x of K elements, as the B operand of the MMAs wants it:
// x = p0 + p1 + p2 exactly (three bf16 parts); the image is [K/16 k-tiles][4 t][4 parts][4 bf16] where
// the four bf16 of (kt, t, part) are elements 16 kt + {2t, 2t+1, 2t+8, 2t+9} of that part -- exactly the
// B fragment (b0, b1) of lane (group = part, t) -- and part 3 is zero.  One 8-byte load per lane per
// k-tile, 128 distinct bytes per warp (lanes of groups 4..7 re-read groups 0..3), no bank conflicts.
__host__ __device__ __forceinline__ int split_pos(int i, int part)
{
    const int c = i & 15, kt = i >> 4;
    const int t = (c & 7) >> 1, j = c & 1, hi = c >> 3;
    return (((kt * 4 + t) * 4 + part) << 2) + 2 * hi + j;
}

__device__ __forceinline__ void store_split(__nv_bfloat16 *split, int i, float x)
{
    const __nv_bfloat16 b0 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(b0);
    const __nv_bfloat16 b1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(b1);
    const __nv_bfloat16 b2 = __float2bfloat16_rn(r2);
    const int pos = split_pos(i, 0);
    split[pos] = b0; split[pos + 4] = b1; split[pos + 8] = b2;
}

// NK consecutive k-tiles (from kt0) of one 16-row tile of a fragment-packed bf16 matrix times a split
// vector.  A: [NKT][32 lanes] uint4.  Straight-line code: all fragment loads are issued before the first
// MMA and the MMAs run back to back over four independent accumulator chains.  D columns 0,1,2 hold the
// products with the three parts of the vector (column 3 is zero, columns 4..7 are repeats that nobody
// reads).  On return the lanes with t = 0 hold the partial totals of rows g (lo) and g + 8 (hi).
template <int NK>
__device__ __forceinline__ void mma_partial(const uint4 *A, int kt0, const __nv_bfloat16 *split, int lane, float &lo, float &hi)
{
    const int g = lane >> 2, t = lane & 3;
    const uint2 *bsrc = reinterpret_cast<const uint2 *>(split) + (kt0 * 4 + t) * 4 + (g & 3);
    const uint4 *a = A + (size_t)kt0 * 32 + lane;
    uint4 av[NK];
    uint2 bv[NK];
#pragma unroll
    for (int i = 0; i < NK; ++i) { av[i] = a[i * 32]; bv[i] = bsrc[16 * i]; }
    float acc[4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[c][i] = 0.f;
#pragma unroll
    for (int i = 0; i < NK; ++i) {
        float *c = acc[i & 3];
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(av[i].x), "r"(av[i].y), "r"(av[i].z), "r"(av[i].w), "r"(bv[i].x), "r"(bv[i].y));
    }
    float s_lo = (acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]) + ((acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]));
    float s_hi = (acc[0][2] + acc[1][2]) + (acc[2][2] + acc[3][2]) + ((acc[0][3] + acc[1][3]) + (acc[2][3] + acc[3][3]));
    s_lo += __shfl_xor_sync(FULL, s_lo, 1);      // t = 0 (columns 0,1) + t = 1 (columns 2,3)
    s_hi += __shfl_xor_sync(FULL, s_hi, 1);
    lo = s_lo; hi = s_hi;
}

// ---------------------------------------------------------------------------------------------
// The same split image with two k-tiles per 16-byte piece: [K/32 k-tile pairs][4 parts][4 t][2 k-tiles][4 bf16], so that
// one 16-byte load per lane brings the B fragments of two k-tiles, the loads of a warp are one contiguous run, and the
// threads that write the image (consecutive elements per lane) spread over the banks.
__host__ __device__ __forceinline__ int split2_pos(int i, int part)
{
    const int c = i & 15, kt = i >> 4;
    const int t = (c & 7) >> 1, j = c & 1, hi = c >> 3;
    return ((((((kt >> 1) * 4 + part) * 4 + t) << 1) + (kt & 1)) << 2) + 2 * hi + j;
}

__device__ __forceinline__ void store_split2(__nv_bfloat16 *split, int i, float x)
{
    const __nv_bfloat16 b0 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(b0);
    const __nv_bfloat16 b1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(b1);
    const __nv_bfloat16 b2 = __float2bfloat16_rn(r2);
    split[split2_pos(i, 0)] = b0; split[split2_pos(i, 1)] = b1; split[split2_pos(i, 2)] = b2;
}
// two adjacent elements (i even): they share a 32-bit word of every part
__device__ __forceinline__ void store_split2_pair(__nv_bfloat16 *split, int i, float x0, float x1)
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
#pragma unroll
    for (int k = 0; k < 3; ++k) s32[split2_pos(i, k) >> 1] = w[k];
}

// NK consecutive k-tiles (NK even, from the even k-tile kt0) of NT 16-row tiles (consecutive in memory, tile_u4 apart) of a
// fragment-packed bf16 matrix times a split2 vector: the B fragments are loaded once for all NT tiles.  On return the
// lanes with t = 0 hold the partial totals of rows g (lo[n]) and g + 8 (hi[n]) of tile n.
template <int NK, int NT>
__device__ __forceinline__ void mma_tiles(const uint4 *A, size_t tile_u4, int kt0, const __nv_bfloat16 *split, int lane, float (&lo)[NT], float (&hi)[NT])
{
    static_assert(NK % 2 == 0, "k-tiles come in pairs");
    const int g = lane >> 2, t = lane & 3;
    const uint4 *bsrc = reinterpret_cast<const uint4 *>(split) + ((kt0 >> 1) * 4 + (g & 3)) * 4 + t;
    uint4 av[NT][NK];
    uint4 bv[NK / 2];
#pragma unroll
    for (int i = 0; i < NK / 2; ++i) bv[i] = bsrc[16 * i];
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
        float s_lo = (acc[n][0][0] + acc[n][1][0]) + (acc[n][0][1] + acc[n][1][1]);
        float s_hi = (acc[n][0][2] + acc[n][1][2]) + (acc[n][0][3] + acc[n][1][3]);
        s_lo += __shfl_xor_sync(FULL, s_lo, 1);      // t = 0 (columns 0,1) + t = 1 (columns 2,3)
        s_hi += __shfl_xor_sync(FULL, s_hi, 1);
        lo[n] = s_lo; hi[n] = s_hi;
    }
}

}  // namespace wrnn
