// Shared device helpers of the attention kernels (bf16 unpacking, streaming loads,
// lane-group reductions, online-softmax state merging).  Internal to the library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bt.h"

namespace bt {

using bf16 = __nv_bfloat16;

constexpr float kNegInf = -__builtin_huge_valf();

// Lanes that share one K or V row: each lane owns 8 consecutive bf16 (one 128-bit load).
template <int HD>
struct RowGeo {
    static_assert(HD == 64 || HD == 128, "head_dim must be 64 or 128");
    static constexpr int LPR = HD / 8;    // lanes per row
    static constexpr int RPW = 32 / LPR;  // rows covered by one warp-wide load
};

// 128-bit read-once load that bypasses L1 allocation (KV rows are streamed exactly once).
__device__ __forceinline__ uint4 ld_stream(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// Plain coherent 128-bit load (for memory this launch may also write).
__device__ __forceinline__ uint4 ld_plain(const void* p) { return *reinterpret_cast<const uint4*>(p); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// bf16 pair packed in a 32-bit word -> two fp32 (exact: bf16 is the top half of fp32).
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ void unpack8(const uint4& r, float (&f)[8])
{
    f[0] = bf_lo(r.x); f[1] = bf_hi(r.x);
    f[2] = bf_lo(r.y); f[3] = bf_hi(r.y);
    f[4] = bf_lo(r.z); f[5] = bf_hi(r.z);
    f[6] = bf_lo(r.w); f[7] = bf_hi(r.w);
}

__device__ __forceinline__ float dot8(const float (&q)[8], const uint4& r)
{
    float a = q[0] * bf_lo(r.x);
    a = fmaf(q[1], bf_hi(r.x), a);
    a = fmaf(q[2], bf_lo(r.y), a);
    a = fmaf(q[3], bf_hi(r.y), a);
    a = fmaf(q[4], bf_lo(r.z), a);
    a = fmaf(q[5], bf_hi(r.z), a);
    a = fmaf(q[6], bf_lo(r.w), a);
    a = fmaf(q[7], bf_hi(r.w), a);
    return a;
}

__device__ __forceinline__ void fma8(float (&acc)[8], float p, const uint4& r)
{
    acc[0] = fmaf(p, bf_lo(r.x), acc[0]); acc[1] = fmaf(p, bf_hi(r.x), acc[1]);
    acc[2] = fmaf(p, bf_lo(r.y), acc[2]); acc[3] = fmaf(p, bf_hi(r.y), acc[3]);
    acc[4] = fmaf(p, bf_lo(r.z), acc[4]); acc[5] = fmaf(p, bf_hi(r.z), acc[5]);
    acc[6] = fmaf(p, bf_lo(r.w), acc[6]); acc[7] = fmaf(p, bf_hi(r.w), acc[7]);
}

// Packed fp32 pairs: one issue slot for two multiply-adds (sm_100).
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t bf2_to_f2(uint32_t w) { return pack2(bf_lo(w), bf_hi(w)); }
// q (4 pairs) . row piece (8 bf16); the two halves of the pairs are added at the end
__device__ __forceinline__ float dot8_x2(const uint64_t (&q2)[4], const uint4& r)
{
    uint64_t a = fmul2(q2[0], bf2_to_f2(r.x));
    a = ffma2(q2[1], bf2_to_f2(r.y), a);
    a = ffma2(q2[2], bf2_to_f2(r.z), a);
    a = ffma2(q2[3], bf2_to_f2(r.w), a);
    float lo, hi;
    unpack2(a, lo, hi);
    return lo + hi;
}
__device__ __forceinline__ void fma8_x2(uint64_t (&acc2)[4], float p, const uint4& r)
{
    const uint64_t p2 = pack2(p, p);
    acc2[0] = ffma2(p2, bf2_to_f2(r.x), acc2[0]);
    acc2[1] = ffma2(p2, bf2_to_f2(r.y), acc2[1]);
    acc2[2] = ffma2(p2, bf2_to_f2(r.z), acc2[2]);
    acc2[3] = ffma2(p2, bf2_to_f2(r.w), acc2[3]);
}

// Sum over the LPR consecutive lanes that hold one row (all of them get the total).
template <int LPR>
__device__ __forceinline__ float row_sum(float x)
{
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

// 8 fp32 -> 8 bf16 (round to nearest even) packed in a uint4.
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(f[2], f[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]);
    __nv_bfloat162 d = __floats2bfloat162_rn(f[6], f[7]);
    uint4 r;
    r.x = *reinterpret_cast<uint32_t*>(&a);
    r.y = *reinterpret_cast<uint32_t*>(&b);
    r.z = *reinterpret_cast<uint32_t*>(&c);
    r.w = *reinterpret_cast<uint32_t*>(&d);
    return r;
}

// Running softmax state of one lane: maximum m (log2 domain), sum l of 2^(s-m), and the
// 8 weighted-value accumulators the lane owns.
struct SoftmaxState {
    float m, l, acc[8];
    __device__ __forceinline__ void init()
    {
        m = kNegInf;
        l = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    }
    // fold another state (m2, l2, acc2) into this one
    __device__ __forceinline__ void merge(float m2, float l2, const float (&a2)[8])
    {
        float mn = fmaxf(m, m2);
        if (mn == kNegInf) return;  // both empty
        float c1 = ex2(m - mn), c2 = ex2(m2 - mn);
        l = l * c1 + l2 * c2;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = acc[i] * c1 + a2[i] * c2;
        m = mn;
    }
};

// Programmatic dependent launch.  A kernel launched with launch_pdl may start while the kernel
// before it in the stream is still draining: it calls pdl_launch_dependents() first (its own
// successor may then be scheduled as soon as SM resources free up) and pdl_wait() before its first
// access to global memory - the wait returns once the preceding kernel has completed and its
// writes are visible, so the kernel sees exactly what ordinary stream order would show it.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ void raise_status(uint32_t* dev_status, uint32_t bits)
{
    if (dev_status && bits) atomicOr(dev_status, bits);
}

}  // namespace bt
