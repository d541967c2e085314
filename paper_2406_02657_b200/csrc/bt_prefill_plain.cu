// Block-decoder prefill on the CUDA cores (paper section 2.3: the block decoder is causal over blocks):
// one query block per CTA over rows 0..t, 128-bit read-once loads, online softmax per lane.  It serves
// the shapes the tensor-core kernel does not take, and as its cross-check.
#include "bt_common.cuh"
#include "bt_kernels.h"

namespace bt {

constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kUnroll = 8;  // independent K (and V) loads in flight per lane

// Attention of one query over rows [r0, r1) of one (b,h) slab, by one CTA of kDecodeWarps
// warps.  On return, threads 0..LPR-1 of warp 0 hold the merged state for their 8 dims
// (st.acc un-normalised, st.m, st.l identical on those lanes).
template <int HD>
__device__ __forceinline__ void attend_range(const bf16* __restrict__ qrow, const bf16* __restrict__ Kb,
                                             const bf16* __restrict__ Vb, int r0, int r1, float scale_log2,
                                             SoftmaxState& st, float* smem /* kDecodeWarps*(HD+2) floats */)
{
    constexpr int LPR = RowGeo<HD>::LPR, RPW = RowGeo<HD>::RPW;
    constexpr int TILE = kUnroll * RPW;  // rows per warp iteration
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, rg = lane / LPR;

    float qf[8];
    {
        uint4 qr = ld_plain(qrow + sub * 8);
        unpack8(qr, qf);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[i] *= scale_log2;
    }
    st.init();

    for (int base = r0 + warp * TILE; base < r1; base += kDecodeWarps * TILE) {
        uint4 kr[kUnroll], vr[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            int row = base + u * RPW + rg;
            kr[u] = (row < r1) ? ld_stream(Kb + (size_t)row * HD + sub * 8) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            int row = base + u * RPW + rg;
            vr[u] = (row < r1) ? ld_stream(Vb + (size_t)row * HD + sub * 8) : make_uint4(0, 0, 0, 0);
        }
        float s[kUnroll];
        float mt = kNegInf;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float d = row_sum<LPR>(dot8(qf, kr[u]));
            int row = base + u * RPW + rg;
            s[u] = (row < r1) ? d : kNegInf;
            mt = fmaxf(mt, s[u]);
        }
        if (mt != kNegInf) {  // uniform within the LPR lanes of a row group
            float mn = fmaxf(st.m, mt);
            float c = ex2(st.m - mn);
            st.l *= c;
#pragma unroll
            for (int i = 0; i < 8; ++i) st.acc[i] *= c;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                float p = ex2(s[u] - mn);
                st.l += p;
                fma8(st.acc, p, vr[u]);
            }
            st.m = mn;
        }
    }

    // merge the RPW row groups of the warp
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, st.m, off);
        float l2 = __shfl_xor_sync(0xffffffffu, st.l, off);
        float a2[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) a2[i] = __shfl_xor_sync(0xffffffffu, st.acc[i], off);
        st.merge(m2, l2, a2);
    }
    // merge the warps through shared memory
    if (rg == 0) {
        float* w = smem + warp * (HD + 2);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[sub * 8 + i] = st.acc[i];
        if (sub == 0) {
            w[HD] = st.m;
            w[HD + 1] = st.l;
        }
    }
    __syncthreads();
    if (warp == 0 && rg == 0) {
#pragma unroll
        for (int w2 = 1; w2 < kDecodeWarps; ++w2) {
            const float* w = smem + w2 * (HD + 2);
            float a2[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) a2[i] = w[sub * 8 + i];
            st.merge(w[HD], w[HD + 1], a2);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Plain prefill: query block t of (b,h) is a decode over rows 0..t (paper section 2.3: the
// block decoder is causal over blocks).  One CTA per (b,h,t).  Correct for any T; the
// tensor-core kernel replaces it for the shapes it supports.
template <int HD>
__global__ void __launch_bounds__(kDecodeThreads) block_prefill_simple_kernel(PrefillArgs a)
{
    constexpr int LPR = RowGeo<HD>::LPR;
    __shared__ float smem[kDecodeWarps * (HD + 2)];
    const int bh = blockIdx.x / a.T, t = blockIdx.x - bh * a.T;
    const bf16* Kb = reinterpret_cast<const bf16*>(a.k) + (size_t)bh * a.kv_seq_stride * HD;
    const bf16* Vb = reinterpret_cast<const bf16*>(a.v) + (size_t)bh * a.kv_seq_stride * HD;
    const size_t qoff = ((size_t)bh * a.T + t) * HD;
    SoftmaxState st;
    attend_range<HD>(reinterpret_cast<const bf16*>(a.q) + qoff, Kb, Vb, 0, t + 1, a.scale_log2, st, smem);
    if (threadIdx.x < LPR) {
        float o[8];
        float inv = 1.f / st.l;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = st.acc[i] * inv;
        *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.out) + qoff + threadIdx.x * 8) = pack8(o);
    }
}

cudaError_t launch_block_prefill_simple(const PrefillArgs& a, cudaStream_t stream)
{
    const long long ctas = (long long)a.B * a.H * a.T;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (a.hd == 64)
        block_prefill_simple_kernel<64><<<(unsigned)ctas, kDecodeThreads, 0, stream>>>(a);
    else
        block_prefill_simple_kernel<128><<<(unsigned)ctas, kDecodeThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace bt
