// The linear maps either side of the attention path, y = W x + b on the 5th-generation tensor cores:
//   - prefix projection (paper section 2.4; appendix on token-decoder variants, "Prefix"): the
//     context embedding of a block is projected into P prefix token embeddings;
//   - QKV projection whose epilogue is the cache append (sections 2.1, 2.3, 2.4: the K,V a layer
//     computes from its input are cached): the Q part goes out as [B][H][n][hd] for the attention
//     call, the K and V parts are written straight to rows len[b] .. len[b]+n-1 of the block or
//     local cache, so no separate append pass touches them.
//
// One persistent CTA per SM, warp-specialised:
//   warps 0-7       : epilogue - thread = accumulator row (= tensor-memory lane), two warps per lane quarter
//                     taking alternate 64-column pieces.  64 columns at a time:
//                     tensor memory -> registers, + bias, -> bf16, through a per-warp swizzled
//                     shared-memory patch so that the global stores are whole 128-byte lines (8 lanes
//                     per row piece: one head of one cache row at head_dim 64), then to q / the cache /
//                     the plain [M][N] output
//   warp 8 (1 lane) : TMA producer - x tile [128 x 64] and W tile [BN x 64] per stage, 128-byte swizzle
//   warp 9 (1 lane) : tcgen05.mma issuer - 128 x BN x 16 instructions, fp32 accumulators in tensor
//                     memory, double-buffered so that the epilogue of a tile runs under the next
//                     tile's products
// BN (64, 128 or 256 output features per tile) is chosen per launch so that there are enough tiles
// for every SM.  Every wait is bounded in wall time and raises BT_DEV_TIMEOUT when it runs out.
//
// Large products run the same kernel on pairs of CTAs (kCtas = 2, a cluster of two SMs, tcgen05 cta_group::2):
// a pair owns a 256 x BN tile, each CTA loads its own 128 rows of x and only HALF of the W tile (its BN/2
// output features) with plain TMA loads - no multicast - that report to the leader CTA's barrier; the leader's
// one MMA thread issues 256 x BN x 16 instructions that read both halves of W from the two CTAs' shared
// memory and accumulate each CTA's 128 rows in that CTA's tensor memory; commits are multicast to both CTAs'
// barriers; each CTA drains its own accumulator and reports to the leader.  Per CTA this moves a third less
// operand data from L2 into shared memory for the same products.
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
constexpr int kEpilogueWarps = 8, kProducerWarp = 8, kMmaWarp = 9;
constexpr int kThreads = 320;
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kSpinLimit = 1u << 26;
constexpr uint64_t kWaitLimitNs = 1000000000ull;  // 1 s: far beyond any legitimate wait
constexpr uint32_t kPatchBytes = 32 * 128;         // per epilogue warp: 32 rows x 64 bf16

constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;   // clears the bit that tells the two CTAs of a pair apart in a shared::cluster address

template <int BN, int kCtas>
struct Cfg {
    static constexpr uint32_t kBBytes = (BN / kCtas) * BK * 2;   // a CTA of a pair holds half of the W tile
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = kStageBytes == 48 * 1024 ? 4 : (kStageBytes == 32 * 1024 ? 6 : 8);
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

// ---- the forms that differ between one CTA and a pair
template <int kCtas>
__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols)
{
    if constexpr (kCtas == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {   // issued by the same warp of both CTAs of the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int kCtas>
__device__ __forceinline__ void tmem_dealloc(uint32_t tmem, uint32_t cols)
{
    if constexpr (kCtas == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
}
// TMA load of a pair's CTA: lands in this CTA's shared memory, reports its bytes to the barrier named by a
// shared::cluster address (the leader's).  No multicast.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void mma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    const uint32_t z = 0;   // no output lane disabled
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z)
        : "memory");
}
// arrives, once the MMAs issued so far are done, on the barrier at this address in both CTAs of the pair
__device__ __forceinline__ void mma_commit_pair(uint32_t bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

template <int BN, int kCtas>
__global__ void __launch_bounds__(kThreads, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW, Params p)
{
    using C = Cfg<BN, kCtas>;
    constexpr int S = C::kStages;
    constexpr uint32_t IDESC = make_idesc(BM * kCtas, BN, false);
    const ProjectArgs& a = p.a;
    // a pair of CTAs works on one tile of 256 rows: `rank` is this CTA's half, `unit` numbers the pairs
    const uint32_t rank = kCtas == 2 ? cluster_cta_rank() : 0u;
    const int unit = (int)blockIdx.x / kCtas, n_units = (int)gridDim.x / kCtas;
    const bool leader = rank == 0;

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
            mbar_init(acc_empty(i), kEpilogueWarps * kCtas);   // the leader's collects both CTAs' epilogue warps
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc<kCtas>(smem_u32(tmem_slot), C::kTmemCols);  // this warp allocates the tensor-memory columns and frees them at the end
    tc_fence_before();
    __syncthreads();
    if constexpr (kCtas == 2) cluster_sync_all();   // the partner's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Programmatic dependent launch: until the kernel before this one in the stream is done, nothing here
    // reads or writes global memory (the descriptor prefetch below touches only the kernel's own parameters).
    pdl_launch_dependents();

    const int n_tiles = p.tiles_m * p.tiles_n;     // tiles of BM * kCtas rows
    const int n_kb = (a.K + BK - 1) / BK;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapX) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapW) : "memory");
            pdl_wait();
            uint32_t it = 0;
            bool ok = true;
            for (int tile = unit; ok && tile < n_tiles; tile += n_units) {
                const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % S;
                    ok = wait(empty(s), ((it / S) & 1) ^ 1, abort_flag, a.dev_status);
                    if (!ok) break;
                    const uint32_t dst = base + s * C::kStageBytes;
                    if constexpr (kCtas == 1) {
                        mbar_expect_tx(full(s), C::kStageBytes);
                        tma_load_3d(dst, &mapX, full(s), kb * BK, tm * BM, 0);
                        tma_load_3d(dst + kABytes, &mapW, full(s), kb * BK, tn * BN, 0);
                    } else {
                        // both CTAs' bytes are counted on the leader's barrier, which the leader arms
                        if (leader) mbar_expect_tx(full(s), 2 * C::kStageBytes);
                        const uint32_t bar = full(s) & kPeerBitMask;
                        tma_load_3d_pair(dst, &mapX, bar, kb * BK, tm * (2 * BM) + (int)rank * BM, 0);
                        tma_load_3d_pair(dst + kABytes, &mapW, bar, kb * BK, tn * BN + (int)rank * (BN / 2), 0);
                    }
                }
            }
            // Before the CTA goes, nothing may still be on its way to it.  One CTA: every copy this thread issued
            // has landed (at once on the normal path, where the products that consumed them are done).  A pair:
            // the last commits multicast to this CTA's "stage free" barriers have arrived, which also means the
            // products that read this CTA's shared memory are done.  Bounded when something went wrong.
            for (uint32_t back = 1; back <= (uint32_t)S && back <= it; ++back) {
                const uint32_t u = it - back;
                if constexpr (kCtas == 1) {
                    if (!mbar_wait_walltime(full(u % S), (u / S) & 1, abort_flag, kSpinLimit, kWaitLimitNs)) break;
                } else {
                    if (!mbar_wait_walltime(empty(u % S), (u / S) & 1, abort_flag, kSpinLimit, kWaitLimitNs)) break;
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // The whole warp walks the loop (control flow stays warp-uniform; the outcome of every wait is agreed on by
        // a vote) and one elected lane issues: a lone lane inside a divergent branch issues tcgen05.mma slower.
        if (leader) {   // a pair's products are issued by its leader alone
            auto wait_all = [&](uint32_t b, uint32_t parity) { return __all_sync(0xffffffffu, wait(b, parity, abort_flag, a.dev_status)) != 0; };
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = unit; ok && tile < n_tiles; tile += n_units, ++t) {
                const uint32_t acc = t & 1;
                ok = wait_all(acc_empty(acc), ((t >> 1) & 1) ^ 1);  // the epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % S;
                    ok = wait_all(full(s), (it / S) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    // descriptor low words: address in 16-byte units plus the leading-dimension field; 16 elements
                    // of K are 32 bytes inside a swizzled 128-byte row
                    const uint32_t a0 = base + s * C::kStageBytes, b0 = a0 + kABytes;
                    const uint32_t alo = (a0 >> 4) | (1u << 16), blo = (b0 >> 4) | (1u << 16);
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            if constexpr (kCtas == 1)
                                mma_bf16(tmem + acc * BN, desc_words(alo + kk * 2, kDescHiSw128), desc_words(blo + kk * 2, kDescHiSw128), IDESC,
                                         (kb > 0 || kk > 0) ? 1u : 0u);
                            else
                                mma_bf16_pair(tmem + acc * BN, desc_words(alo + kk * 2, kDescHiSw128), desc_words(blo + kk * 2, kDescHiSw128), IDESC,
                                              (kb > 0 || kk > 0) ? 1u : 0u);
                        }
                        if constexpr (kCtas == 1) mma_commit(empty(s));
                        else mma_commit_pair(empty(s));
                        if (kb == n_kb - 1) {
                            if constexpr (kCtas == 1) mma_commit(acc_full(acc));
                            else mma_commit_pair(acc_full(acc));
                        }
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: thread = output row
        // warps 0-7: warp e drains tensor-memory lane quarter e % 4 (the quarter a warp may access is its index
        // modulo 4) and every other 64-column piece, starting at piece e / 4
        const int wq = warp & 3, half = warp >> 2;
        const uint32_t lane_base = tmem + ((uint32_t)(wq * 32) << 16);
        const uint32_t patch = sPatch + warp * kPatchBytes;
        const bf16* bias = reinterpret_cast<const bf16*>(a.bias);
        const int D = a.H * a.hd;
        uint32_t t = 0;
        bool ok = true;
        pdl_wait();
        for (int tile = unit; tile < n_tiles; tile += n_units, ++t) {
            const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
            const uint32_t acc = t & 1;
            // this lane's own row: which sequence, which of its n rows, and where the row lands in the cache
            const int m = tm * (BM * kCtas) + (int)rank * BM + wq * 32 + lane;
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
            for (int c0 = half * 64; c0 < BN; c0 += 128) {
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
            if (lane == 0) {
                if constexpr (kCtas == 1) mbar_arrive(acc_empty(acc));
                else mbar_arrive_cluster(acc_empty(acc) & kPeerBitMask);   // the leader's barrier
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (kCtas == 2) cluster_sync_all();   // both CTAs are through with each other's barriers and tensor memory
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc<kCtas>(tmem, C::kTmemCols);
    }
}

// The lengths go up once every tile has read the old ones: a second, tiny launch behind the product (it starts
// under programmatic dependent launch while the product drains; counting the product's CTAs in on a word in
// global memory and letting the last one advance the lengths was measured 2 us slower per step).
__global__ void project_len_advance_kernel(int32_t* len, int B, int n, int cap, int reset_first, const uint8_t* reset_mask,
                                           uint32_t* dev_status)
{
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) advance_len(len, b, n, cap, reset_first, reset_mask, dev_status);
}

template <int BN, int kCtas>
static cudaError_t launch_bn(const ProjectArgs& a, int dev, int sms, cudaStream_t stream)
{
    using C = Cfg<BN, kCtas>;
    static PerDeviceOnce limit_raised;
    cudaError_t e = raise_smem_limit_once(limit_raised, dev, project_tc_kernel<BN, kCtas>, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap mx, mw;
    if (!make_slab_map(&mx, a.x, a.K, a.M, a.M, 1, BM) || !make_slab_map(&mw, a.w, a.K, a.N, a.N, 1, BN / kCtas)) return cudaErrorInvalidValue;
    Params p;
    p.a = a;
    p.tiles_m = (a.M + BM * kCtas - 1) / (BM * kCtas);
    p.tiles_n = (a.N + BN - 1) / BN;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int units = sms / kCtas;
    const int grid = (int)(tiles < units ? tiles : units) * kCtas;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)C::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kCtas;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = kCtas == 2 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, project_tc_kernel<BN, kCtas>, mx, mw, p);
}

}  // namespace proj

bool project_supported(const ProjectArgs& a) { return a.K % 8 == 0 && a.N % 8 == 0 && tensor_map_encode_fn() != nullptr; }

cudaError_t launch_project(const ProjectArgs& a, cudaStream_t stream)
{
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    // Tile shape: the one with the shortest estimated launch.  All tiles of a launch take the same time, so a launch
    // lasts (rounds of tiles) x (time of one tile); a tile's time is its area per SM over the relative rate that
    // shape sustains (measured: 128 x 256 on one SM = 1; 256 x 256 on a pair 1.11, a third less operand traffic per
    // SM; the narrower tiles less, their operands being re-read more often).
    struct Shape {
        int bn, ctas;
        double rate;
    };
    const Shape shapes[4] = {{256, 2, 1.11}, {256, 1, 1.0}, {128, 1, 0.9}, {64, 1, 0.75}};
    int best = 1;
    double best_cost = 0.0;
    for (int i = 0; i < 4; ++i) {
        const Shape& sh = shapes[i];
        if (sh.ctas == 2 && sms % 2 != 0) continue;
        const long long rows = (long long)proj::BM * sh.ctas;
        const long long tiles = ((a.M + rows - 1) / rows) * ((a.N + sh.bn - 1) / sh.bn);
        const long long units = sms / sh.ctas;
        const long long rounds = (tiles + units - 1) / units;
        const double cost = (double)rounds * (double)(proj::BM * sh.bn) / sh.rate;
        if (i == 0 || cost < best_cost - 1e-9) {
            best = i;
            best_cost = cost;
        }
    }
    switch (best) {
        case 0: e = proj::launch_bn<256, 2>(a, dev, sms, stream); break;
        case 1: e = proj::launch_bn<256, 1>(a, dev, sms, stream); break;
        case 2: e = proj::launch_bn<128, 1>(a, dev, sms, stream); break;
        default: e = proj::launch_bn<64, 1>(a, dev, sms, stream); break;
    }
    if (e != cudaSuccess || a.mode == kProjectPlain) return e;
    const int B = a.M / a.n_rows;
    return launch_pdl(proj::project_len_advance_kernel, dim3((B + 255) / 256), dim3(256), 0, stream, a.cache.len, B, a.n_rows,
                      a.cache.cap, a.reset_first, a.reset_mask, a.dev_status);
}

}  // namespace bt
