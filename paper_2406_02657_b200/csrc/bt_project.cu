// The linear maps either side of the attention path, y = W x + b on the 5th-generation tensor cores:
//   - prefix projection (paper section 2.4; appendix on token-decoder variants, "Prefix"): the
//     context embedding of a block is projected into P prefix token embeddings;
//   - QKV projection whose epilogue is the cache append (sections 2.1, 2.3, 2.4: the K,V a layer
//     computes from its input are cached): the Q part goes out as [B][H][n][hd] for the attention
//     call, the K and V parts are written straight to rows len[b] .. len[b]+n-1 of the block or
//     local cache, so no separate append pass touches them.
//
// One persistent CTA per SM, warp-specialised:
//   warps 0-3       : epilogue - thread = accumulator row (= tensor-memory lane).  64 columns at a time:
//                     tensor memory -> registers, + bias, -> bf16, through a per-warp swizzled
//                     shared-memory patch so that the global stores are whole 128-byte lines (8 lanes
//                     per row piece: one head of one cache row at head_dim 64), then to q / the cache /
//                     the plain [M][N] output
//   warp 4 (1 lane) : TMA producer - x tile [128 x 64] and W tile [BN x 64] per stage, 128-byte swizzle
//   warp 5 (1 lane) : tcgen05.mma issuer - 128 x BN x 16 instructions, fp32 accumulators in tensor
//                     memory, double-buffered so that the epilogue of a tile runs under the next
//                     tile's products
// BN (64, 128 or 256 output features per tile) is chosen per launch so that there are enough tiles
// for every SM.  Every wait is bounded in wall time and raises BT_DEV_TIMEOUT when it runs out.
#include <cuda.h>

#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"
#include "bt_tcgen05.cuh"
#include "bt_tensor_map.h"

namespace bt {
namespace proj {

using namespace tc;

constexpr int BM = 128;                  // rows of x per tile (= tensor-memory lanes)
constexpr int BK = 64;                   // K elements per stage: one 128-byte swizzle atom
constexpr int kEpilogueWarps = 4, kProducerWarp = 4, kMmaWarp = 5;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kSpinLimit = 1u << 26;
constexpr uint64_t kWaitLimitNs = 1000000000ull;  // 1 s: far beyond any legitimate wait
constexpr uint32_t kPatchBytes = 32 * 128;         // per epilogue warp: 32 rows x 64 bf16

template <int BN>
struct Cfg {
    static constexpr uint32_t kBBytes = BN * BK * 2;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr uint32_t kTmemCols = 2 * BN;   // two accumulators
    static constexpr int kBarriers = 2 * kStages + 4;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kEpilogueWarps * kPatchBytes + kBarriers * 8 + 16;
};

struct Params {
    ProjectArgs a;
    int tiles_m, tiles_n;
};

__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* dev_status)
{
    if (mbar_wait_walltime(bar, parity, abort_flag, kSpinLimit, kWaitLimitNs)) return true;
    raise_status(dev_status, BT_DEV_TIMEOUT);
    return false;
}

// New length of sequence b after its n rows: (reset ? 0 : len) + n when they fit, else unchanged and flagged.
__device__ __forceinline__ void advance_len(int32_t* len, int b, int n, int cap, int reset_first, const uint8_t* reset_mask,
                                            uint32_t* dev_status)
{
    const bool rst = reset_mask ? (reset_mask[b] != 0) : (reset_first != 0);
    const int l = rst ? 0 : len[b];
    if (l >= 0 && l + n <= cap)
        len[b] = l + n;
    else
        raise_status(dev_status, BT_DEV_OVERFLOW);  // the sequence keeps its rows and its length
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW, Params p)
{
    using C = Cfg<BN>;
    constexpr int S = C::kStages;
    constexpr uint32_t IDESC = make_idesc(BM, BN, false);
    const ProjectArgs& a = p.a;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sPatch = base + S * C::kStageBytes;
    const uint32_t sBar = sPatch + kEpilogueWarps * kPatchBytes;
    uint8_t* gen_tail = gen_base + (sBar - base);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_tail + C::kBarriers * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_tail + C::kBarriers * 8 + 8);
    auto full = [&](int s) { return sBar + 8u * s; };
    auto empty = [&](int s) { return sBar + 8u * (S + s); };
    auto acc_full = [&](int i) { return sBar + 8u * (2 * S + i); };
    auto acc_empty = [&](int i) { return sBar + 8u * (2 * S + 2 + i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full(s), 1);
            mbar_init(empty(s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(acc_full(i), 1);
            mbar_init(acc_empty(i), kEpilogueWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // this warp allocates the CTA's tensor-memory columns and frees them at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Programmatic dependent launch: until the kernel before this one in the stream is done, nothing here
    // reads or writes global memory (the descriptor prefetch below touches only the kernel's own parameters).
    pdl_launch_dependents();

    const int n_tiles = p.tiles_m * p.tiles_n;
    const int n_kb = (a.K + BK - 1) / BK;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapX) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapW) : "memory");
            pdl_wait();
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
                const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % S;
                    ok = wait(empty(s), ((it / S) & 1) ^ 1, abort_flag, a.dev_status);
                    if (!ok) break;
                    const uint32_t dst = base + s * C::kStageBytes;
                    mbar_expect_tx(full(s), C::kStageBytes);
                    tma_load_3d(dst, &mapX, full(s), kb * BK, tm * BM, 0);
                    tma_load_3d(dst + kABytes, &mapW, full(s), kb * BK, tn * BN, 0);
                }
            }
            // before the CTA goes: every copy this thread issued has landed (at once on the normal path, where the
            // products that consumed them are done; bounded when something went wrong)
            for (uint32_t back = 1; back <= (uint32_t)S && back <= it; ++back) {
                const uint32_t u = it - back;
                if (!mbar_wait_walltime(full(u % S), (u / S) & 1, abort_flag, kSpinLimit, kWaitLimitNs)) break;
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane == 0) {
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++t) {
                const uint32_t acc = t & 1;
                ok = wait(acc_empty(acc), ((t >> 1) & 1) ^ 1, abort_flag, a.dev_status);  // the epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % S;
                    ok = wait(full(s), (it / S) & 1, abort_flag, a.dev_status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a0 = base + s * C::kStageBytes, b0 = a0 + kABytes;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        mma_bf16(tmem + acc * BN, make_desc(a0 + kk * 32, 16, 1024), make_desc(b0 + kk * 32, 16, 1024), IDESC,
                                 (kb > 0 || kk > 0) ? 1u : 0u);
                    mma_commit(empty(s));
                }
                if (ok) mma_commit(acc_full(acc));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: thread = output row
        const int wq = warp;                                   // warps 0-3: tensor-memory lane quarter
        const uint32_t lane_base = tmem + ((uint32_t)(wq * 32) << 16);
        const uint32_t patch = sPatch + wq * kPatchBytes;
        const bf16* bias = reinterpret_cast<const bf16*>(a.bias);
        const int D = a.H * a.hd;
        uint32_t t = 0;
        bool ok = true;
        pdl_wait();
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++t) {
            const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
            const uint32_t acc = t & 1;
            // this lane's own row: which sequence, which of its n rows, and where the row lands in the cache
            const int m = tm * BM + wq * 32 + lane;
            int row_b = -1, row_i = 0, row_rc = -1;
            if (m < a.M) {
                if (a.mode == kProjectPlain) {
                    row_b = m;
                } else {
                    row_b = m / a.n_rows;
                    row_i = m - row_b * a.n_rows;
                    const bool rst = a.reset_mask ? (a.reset_mask[row_b] != 0) : (a.reset_first != 0);
                    const int len_old = rst ? 0 : a.cache.len[row_b];
                    if (len_old >= 0 && len_old + a.n_rows <= a.cache.cap) row_rc = len_old + row_i;  // else: no room, K and V are dropped
                }
            }
            ok = wait(acc_full(acc), (t >> 1) & 1, abort_flag, a.dev_status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 64) {
                const int col0 = tn * BN + c0;                 // first output feature of this 64-column piece
                if (col0 >= a.N) break;                        // warp-uniform
                uint32_t r[64];
                tmem_ld32_issue(lane_base + acc * BN + c0, r);
                tmem_ld32_issue(lane_base + acc * BN + c0 + 32, r + 32);
                tmem_wait_ld();
                tmem_ld_fence32(r);
                tmem_ld_fence32(r + 32);
                // + bias, -> bf16, into the patch: row `lane`, 16-byte piece q8 at (q8 ^ (lane & 7))
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(r[q8 * 8 + i]);
                    const int col = col0 + q8 * 8;
                    if (bias != nullptr && col < a.N) {
                        float bf[8];
                        unpack8(*reinterpret_cast<const uint4*>(bias + col), bf);
#pragma unroll
                        for (int i = 0; i < 8; ++i) f[i] += bf[i];
                    }
                    const uint4 w = pack8(f);
                    const uint32_t dst = patch + lane * 128 + ((q8 ^ (lane & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
                }
                __syncwarp();
                // Where the piece goes.  head_dim is a multiple of 64 and so is col0: the 64 columns lie inside one
                // head of one of Q, K, V, so everything but the row is the same for the whole warp.
                bf16* piece_base = reinterpret_cast<bf16*>(a.out);
                size_t slab_elems = 0, row_elems = 0;     // element strides: per (sequence, head) slab, per row
                int piece_h = 0, piece_d = 0;
                bool to_cache = false;
                if (a.mode == kProjectQkv) {
                    const int part = col0 / D, cc = col0 - part * D;   // 0: Q, 1: K, 2: V
                    piece_h = cc / a.hd;
                    piece_d = cc - piece_h * a.hd;
                    to_cache = part != 0;
                    if (to_cache) {
                        piece_base = reinterpret_cast<bf16*>(part == 1 ? a.cache.k : a.cache.v);
                        slab_elems = (size_t)a.cache.slab_stride;
                        row_elems = (size_t)a.cache.row_stride;
                    } else {
                        slab_elems = (size_t)a.n_rows * a.hd;
                        row_elems = (size_t)a.hd;
                    }
                }
                // out of the patch: 8 lanes take one row's 128 bytes, so every store instruction writes 4 whole lines
#pragma unroll
                for (int itr = 0; itr < 8; ++itr) {
                    const int rr = itr * 4 + (lane >> 3), q8 = lane & 7;
                    const int b = __shfl_sync(0xffffffffu, row_b, rr);
                    const int i = __shfl_sync(0xffffffffu, row_i, rr);
                    const int rc = __shfl_sync(0xffffffffu, row_rc, rr);
                    uint4 w;
                    const uint32_t src = patch + rr * 128 + ((q8 ^ (rr & 7)) << 4);
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(src) : "memory");
                    const int col = col0 + q8 * 8;
                    if (b < 0 || col >= a.N) continue;
                    bf16* dst = nullptr;
                    if (a.mode == kProjectPlain)
                        dst = piece_base + (size_t)b * a.N + col;
                    else if (!to_cache || rc >= 0)   // Q row i of the sequence, or cache row rc (absent when there is no room)
                        dst = piece_base + ((size_t)b * a.H + piece_h) * slab_elems + (size_t)(to_cache ? rc : i) * row_elems + piece_d + q8 * 8;
                    if (dst) *reinterpret_cast<uint4*>(dst) = w;
                }
                __syncwarp();  // the patch is free for the next piece
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(acc));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
    }
    // With a sync word the lengths go up inside this launch: every CTA counts itself in once all of its tiles are
    // stored (the barrier above: all epilogue warps are through), and the one that arrives last - when nobody
    // reads the old lengths any more - advances them and puts the word back to zero.
    if (a.mode == kProjectQkv && a.sync_word != nullptr) {
        __shared__ int is_last;
        if (threadIdx.x == 0) {
            __threadfence();
            is_last = atomicAdd(a.sync_word, 1u) == gridDim.x - 1;
        }
        __syncthreads();
        if (is_last) {
            pdl_wait();  // not every thread of the CTA has been through it yet
            __threadfence();
            const int B = a.M / a.n_rows;
            for (int b = threadIdx.x; b < B; b += blockDim.x) advance_len(a.cache.len, b, a.n_rows, a.cache.cap, a.reset_first, a.reset_mask, a.dev_status);
            if (threadIdx.x == 0) *a.sync_word = 0u;
        }
    }
}

// The lengths go up once every tile has read the old ones: without a sync word, a second, tiny launch
// behind the product.
__global__ void project_len_advance_kernel(int32_t* len, int B, int n, int cap, int reset_first, const uint8_t* reset_mask,
                                           uint32_t* dev_status)
{
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) advance_len(len, b, n, cap, reset_first, reset_mask, dev_status);
}

template <int BN>
static cudaError_t launch_bn(const ProjectArgs& a, int dev, int sms, cudaStream_t stream)
{
    using C = Cfg<BN>;
    static PerDeviceOnce limit_raised;
    cudaError_t e = raise_smem_limit_once(limit_raised, dev, project_tc_kernel<BN>, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap mx, mw;
    if (!make_slab_map(&mx, a.x, a.K, a.M, a.M, 1, BM) || !make_slab_map(&mw, a.w, a.K, a.N, a.N, 1, BN)) return cudaErrorInvalidValue;
    Params p;
    p.a = a;
    p.tiles_m = (a.M + BM - 1) / BM;
    p.tiles_n = (a.N + BN - 1) / BN;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int grid = (int)(tiles < sms ? tiles : sms);
    return launch_pdl(project_tc_kernel<BN>, dim3(grid), dim3(kThreads), (size_t)C::kSmemBytes, stream, mx, mw, p);
}

}  // namespace proj

bool project_supported(const ProjectArgs& a) { return a.K % 8 == 0 && a.N % 8 == 0 && tensor_map_encode_fn() != nullptr; }

cudaError_t launch_project(const ProjectArgs& a, cudaStream_t stream)
{
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    // the widest tile that still gives every SM one
    const long long tiles_m = (a.M + proj::BM - 1) / proj::BM;
    auto tiles = [&](int bn) { return tiles_m * ((a.N + bn - 1) / bn); };
    if (tiles(256) >= sms)
        e = proj::launch_bn<256>(a, dev, sms, stream);
    else if (tiles(128) >= sms)
        e = proj::launch_bn<128>(a, dev, sms, stream);
    else
        e = proj::launch_bn<64>(a, dev, sms, stream);
    if (e != cudaSuccess || a.mode == kProjectPlain || a.sync_word != nullptr) return e;
    const int B = a.M / a.n_rows;
    return launch_pdl(proj::project_len_advance_kernel, dim3((B + 255) / 256), dim3(256), 0, stream, a.cache.len, B, a.n_rows,
                      a.cache.cap, a.reset_first, a.reset_mask, a.dev_status);
}

}  // namespace bt
