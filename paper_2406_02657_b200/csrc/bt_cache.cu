// KV-cache bookkeeping kernels: append rows at the per-sequence length, reset lengths at a
// block boundary (paper sections 2.1, 2.3, 2.4; Figure 1).  Pure index arithmetic and
// 128-bit copies; results are bit-exact by construction.
#include "bt_common.cuh"
#include "bt_kernels.h"

namespace bt {

constexpr int kAppendThreads = 256;

// Copies the rows of sequence b = blockIdx.x.  gridDim.y CTAs share the 16-byte chunks of the
// sequence.  With kFused (gridDim.y == 1) the same CTA also advances len[b]: every thread
// reads the old length before the barrier, one thread writes the new one after it.
template <bool kFused>
__global__ void __launch_bounds__(kAppendThreads) kv_append_kernel(CacheView c, int H, int hd, const bf16* __restrict__ k_new,
                                                                   const bf16* __restrict__ v_new, int n_new,
                                                                   uint32_t* dev_status)
{
    const int b = blockIdx.x;
    if (kFused) {  // launched with launch_pdl
        pdl_launch_dependents();
        // warm L2 with the length and the rows to copy while the kernel before this one drains
        // (a prefetch returns nothing to the thread, so it is safe ahead of the wait)
        if (threadIdx.x == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(c.len + b));
        const size_t bytes = (size_t)H * n_new * hd * 2;
        for (size_t o = (size_t)threadIdx.x * 128; o < bytes; o += (size_t)blockDim.x * 128) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(k_new) + (size_t)b * bytes + o));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(v_new) + (size_t)b * bytes + o));
        }
        pdl_wait();
    }
    const int len = c.len[b];
    if (kFused) __syncthreads();
    const bool ok = len >= 0 && len + n_new <= c.cap;
    if (ok) {
        const int lpr = hd / 8;
        const long long chunks = (long long)H * n_new * lpr;
        bf16* kc = reinterpret_cast<bf16*>(c.k);
        bf16* vc = reinterpret_cast<bf16*>(c.v);
        for (long long idx = (long long)blockIdx.y * blockDim.x + threadIdx.x; idx < chunks;
             idx += (long long)gridDim.y * blockDim.x) {
            const int sub = (int)(idx % lpr);
            const long long hr = idx / lpr;
            const int i = (int)(hr % n_new), h = (int)(hr / n_new);
            const size_t slab = (size_t)b * H + h;
            const size_t src = (slab * n_new + i) * hd + sub * 8;
            const size_t dst = slab * c.slab_stride + (size_t)(len + i) * c.row_stride + sub * 8;
            *reinterpret_cast<uint4*>(kc + dst) = ld_stream(k_new + src);
            *reinterpret_cast<uint4*>(vc + dst) = ld_stream(v_new + src);
        }
    }
    if (kFused && threadIdx.x == 0) {
        if (ok)
            c.len[b] = len + n_new;
        else
            raise_status(dev_status, BT_DEV_OVERFLOW);
    }
}

// Second half of the unfused append: advance the lengths once all rows are in place.
__global__ void len_advance_kernel(int32_t* len, int B, int n_new, int cap, uint32_t* dev_status)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int l = len[b];
    if (l >= 0 && l + n_new <= cap)
        len[b] = l + n_new;
    else
        raise_status(dev_status, BT_DEV_OVERFLOW);
}

__global__ void len_reset_kernel(int32_t* len, int B, const uint8_t* mask)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B && (!mask || mask[b])) len[b] = 0;
}

cudaError_t launch_kv_append(const CacheView& c, int B, int H, int hd, const void* k_new, const void* v_new,
                             int n_new, uint32_t* dev_status, cudaStream_t stream)
{
    const long long chunks = (long long)H * n_new * (hd / 8);
    const bf16* kn = reinterpret_cast<const bf16*>(k_new);
    const bf16* vn = reinterpret_cast<const bf16*>(v_new);
    if (chunks <= 4 * kAppendThreads) {
        return launch_pdl(kv_append_kernel<true>, dim3(B, 1), dim3(kAppendThreads), 0, stream, c, H, hd, kn, vn, n_new, dev_status);
    }
    long long gy = (chunks + 4 * kAppendThreads - 1) / (4 * kAppendThreads);
    if (gy > 1024) gy = 1024;
    kv_append_kernel<false><<<dim3(B, (unsigned)gy), kAppendThreads, 0, stream>>>(c, H, hd, kn, vn, n_new, dev_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    len_advance_kernel<<<(B + 255) / 256, 256, 0, stream>>>(c.len, B, n_new, c.cap, dev_status);
    return cudaGetLastError();
}

cudaError_t launch_len_reset(int32_t* len, int B, const uint8_t* mask, cudaStream_t stream)
{
    len_reset_kernel<<<(B + 255) / 256, 256, 0, stream>>>(len, B, mask);
    return cudaGetLastError();
}

}  // namespace bt
