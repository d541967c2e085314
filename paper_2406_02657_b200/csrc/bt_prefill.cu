// Block-decoder prefill attention on the 5th-generation tensor cores (paper sections 2.1, 2.3:
// the prefill stage processes all prompt blocks in parallel; causal over blocks).
//
// Persistent kernel, one CTA per SM (all of its shared memory and its 512 tensor-memory columns).
// A work item is a pair of neighbouring 128-row query tiles of one (sequence, head); the two tiles
// walk the same key/value tiles 0 .. diagonal, so K and V are loaded once for both.  Roles:
//   warps 0-3 / 4-7 : softmax of query tile A / B - each thread owns one query row (= one TMEM lane)
//                     and holds its 128 scores in registers: one batch of tensor-memory loads, row
//                     maximum, exp2 (packed fp32x2 multiply-adds around it), bf16 P written over the S
//                     columns (signalled in two parts), running row sum; on the diagonal tile a warp
//                     skips the column chunks that are masked for all of its rows.  O is rescaled in
//                     TMEM only when the row maximum grew by more than 2^8 (otherwise the old
//                     reference is kept, exact because O and the row sum share it).  At the end of an
//                     item the rows go through shared memory (the stage of the tile's last V tile)
//                     to a TMA store.
//   warp 8 (1 lane) : TMA producer - Q tiles (Q_A double-buffered an item ahead), K and V rings of
//                     two stages, 128-byte swizzle
//   warp 9 (1 lane) : tcgen05.mma issuer - S = Q K^T into tensor memory, O += P V with P read from
//                     tensor memory (the probabilities never visit shared memory), in the order
//                     PV_A(j) S_A(j+1) PV_B(j) S_B(j+1): the tensor pipe works for one tile while the
//                     other tile is in its softmax
// All waits are bounded in wall time: one that runs out raises BT_DEV_TIMEOUT and the CTA winds down.
#include <cuda.h>

#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"
#include "bt_tcgen05.cuh"
#include "bt_tensor_map.h"

namespace bt {
namespace pf {

constexpr int BM = 128;             // query rows per CTA
constexpr int BN = 128;             // key/value rows per tile
constexpr int kBoxBytes = 128 * 128;  // one TMA box: 128 rows x 64 bf16 (128 bytes, swizzled)
constexpr uint32_t kSpinLimit = 1u << 26;
constexpr uint64_t kWaitLimitNs = 1000000000ull;  // 1 s: far beyond any legitimate wait
constexpr float kRescaleThreshold = 8.0f;  // log2 units

// Bounded wait: gives up after kWaitLimitNs of wall time (or kSpinLimit polls).  Returns false when
// the limit ran out (BT_DEV_TIMEOUT is raised) or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* dev_status)
{
    if (mbar_wait_walltime(bar, parity, abort_flag, kSpinLimit, kWaitLimitNs)) return true;
    raise_status(dev_status, BT_DEV_TIMEOUT);
    return false;
}

using namespace tc;

// Packed fp32 pairs (one issue slot for two lanes' worth of work on sm_100).
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
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Work decomposition.  The T query blocks of one (sequence, head) form n = ceil(T/128) query tiles;
// tile t needs key/value tiles 0..t.  An item is a pair of neighbouring query tiles taken from the
// top: class k holds tiles A = n-1-2k (na = n-2k tile steps) and B = n-2-2k (nb = na-1 steps; absent
// when A is tile 0).  The two tiles of an item walk the same key/value tiles, so K and V are loaded
// once for both and their work is nearly equal, which keeps both softmax warpgroups busy.
// Items are numbered item = bh * m + k (m = ceil(n/2) classes) and CTA c processes items c, c+G,
// c+2G, ... with the grid size G coprime to m, so every CTA cycles through all classes (balanced
// work) while the classes of one (sequence, head) run at the same time on neighbouring CTAs and
// share its K and V through L2.
struct Params {
    uint32_t* dev_status;
    int T, n_qtiles, n_classes;
    long long n_items;
    float scale_log2;
};

// warps 0-3: softmax warpgroup of tile A, warps 4-7: of tile B
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kThreads = 320;
constexpr int kKvStages = 2;
#ifndef BT_PF_EARLY_CHUNKS
#define BT_PF_EARLY_CHUNKS 3
#endif
constexpr int kEarlyChunks = BT_PF_EARLY_CHUNKS;             // 32-column chunks of P signalled ahead of the rest
constexpr int kQBufs = 3;                   // Q_A alternates between buffers 0 and 2, Q_B lives in buffer 1

// barrier slots in shared memory
enum {
    B_QFULL = 0,                       // [kQBufs]  TMA -> MMA
    B_QEMPTY = B_QFULL + kQBufs,       // [kQBufs]  MMA (commit) -> TMA
    B_KFULL = B_QEMPTY + kQBufs,       // [kKvStages]
    B_KEMPTY = B_KFULL + kKvStages,
    B_VFULL = B_KEMPTY + kKvStages,
    B_VEMPTY = B_VFULL + kKvStages,
    B_SFULL = B_VEMPTY + kKvStages,    // [2] per query tile: S ready (and every earlier MMA done)
    B_P0FULL = B_SFULL + 2,            // [2] per query tile: 128 softmax threads have written P columns 0..95
    B_P1FULL = B_P0FULL + 2,           // [2] per query tile: ... and columns 96..127
    B_OFULL = B_P1FULL + 2,            // [2] per query tile: last P V of the item done
    B_COUNT = B_OFULL + 2
};

template <int HD>
constexpr int smem_bytes()
{
    // 3 Q tiles, 2 K and 2 V stages (HD/64 boxes each), barriers, plus 1024 to align
    return 1024 + (HD / 64) * kBoxBytes * (kQBufs + 2 * kKvStages) + 256;
}

constexpr uint32_t kTmemCols = 512;  // S_A, S_B (128 columns each), O_A, O_B (head_dim columns each)

// The class-k item of a (sequence, head) with n query tiles.
struct Item {
    int bh, qa, qb, na, nb;  // qb = -1 and nb = 0 when the item has one tile only
};
__device__ __forceinline__ Item decode_item(long long item, const Params& p)
{
    Item it;
    it.bh = (int)(item / p.n_classes);
    const int k = (int)(item - (long long)it.bh * p.n_classes);
    it.qa = p.n_qtiles - 1 - 2 * k;
    it.qb = it.qa - 1;
    it.na = it.qa + 1;
    it.nb = it.qb + 1;  // 0 when qb == -1
    return it;
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
block_prefill_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO, Params p)
{
    constexpr int NB = HD / 64;                 // TMA boxes per operand tile
    constexpr uint32_t TILE_BYTES = NB * kBoxBytes;
    constexpr uint32_t IDESC_S = make_idesc(BM, BN, false);
    constexpr uint32_t IDESC_O = make_idesc(BM, HD, true);
    // TMEM columns: S (fp32) / P (bf16 pairs, in place) of tiles A and B, then O of tiles A and B
    constexpr uint32_t COL_S0 = 0, COL_O0 = 2 * BN;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sQ = base;                               // kQBufs tiles
    const uint32_t sK = sQ + kQBufs * TILE_BYTES;           // kKvStages tiles
    const uint32_t sV = sK + kKvStages * TILE_BYTES;        // kKvStages tiles
    const uint32_t sBar = sV + kKvStages * TILE_BYTES;      // B_COUNT x 8 bytes
    uint8_t* gen_tail = gen_base + (sBar - base);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_tail + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_tail + B_COUNT * 8 + 8);
    auto bar = [&](int i) { return sBar + 8u * i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(bar(i), (i >= B_P0FULL && i < B_P0FULL + 4) ? 128u : 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // this warp allocates the CTA's tensor-memory columns and frees them at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Programmatic dependent launch: this CTA may have been placed while the kernel before it in the
    // stream drains.  Until that kernel is done only L2 prefetches are issued (they return nothing to
    // the thread): the first item's Q tiles and its first K and V tiles.
    pdl_launch_dependents();
    if (warp == kProducerWarp && lane == 0 && (long long)blockIdx.x < p.n_items) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapQ) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
        const Item it = decode_item(blockIdx.x, p);
        for (int bx = 0; bx < NB; ++bx) {
            tma_prefetch_l2_3d(&mapQ, bx * 64, it.qa * BM, it.bh);
            if (it.nb > 0) tma_prefetch_l2_3d(&mapQ, bx * 64, it.qb * BM, it.bh);
            for (int j = 0; j < it.na && j < kKvStages; ++j) {
                tma_prefetch_l2_3d(&mapK, bx * 64, j * BN, it.bh);
                tma_prefetch_l2_3d(&mapV, bx * 64, j * BN, it.bh);
            }
        }
    }
    pdl_wait();

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapQ) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapO) : "memory");
            // n-th use of a buffer: wait for its EMPTY barrier with parity (n & 1) ^ 1 (passes at once
            // on a fresh barrier), then fill it; the consumer waits FULL with parity n & 1.
            uint32_t q_uses[kQBufs] = {0, 0, 0};
            uint32_t kv_count = 0;   // key/value tiles loaded so far (K and V advance together)
            uint32_t n_done = 0;     // items processed by this CTA
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++n_done) {
                const Item it = decode_item(item, p);
                auto load_q = [&](int buf, int qt) {
                    ok = ok && mbar_wait(bar(B_QEMPTY + buf), (q_uses[buf] & 1) ^ 1, abort_flag, p.dev_status);
                    if (!ok) return;
                    ++q_uses[buf];
                    mbar_expect_tx(bar(B_QFULL + buf), TILE_BYTES);
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sQ + buf * TILE_BYTES + bx * kBoxBytes, &mapQ, bar(B_QFULL + buf), bx * 64, qt * BM, it.bh);
                };
                load_q((n_done & 1) ? 2 : 0, it.qa);
                if (it.nb > 0) load_q(1, it.qb);
                for (int j = 0; ok && j < it.na; ++j, ++kv_count) {
                    const uint32_t st = kv_count % kKvStages, par = ((kv_count / kKvStages) & 1) ^ 1;
                    ok = mbar_wait(bar(B_KEMPTY + st), par, abort_flag, p.dev_status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_KFULL + st), TILE_BYTES);
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sK + st * TILE_BYTES + bx * kBoxBytes, &mapK, bar(B_KFULL + st), bx * 64, j * BN, it.bh);
                    ok = mbar_wait(bar(B_VEMPTY + st), par, abort_flag, p.dev_status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_VFULL + st), TILE_BYTES);
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sV + st * TILE_BYTES + bx * kBoxBytes, &mapV, bar(B_VFULL + st), bx * 64, j * BN, it.bh);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        // Issue order per item (tile A has one more step than tile B):
        //   S_A(0) S_B(0) | PV_A(0) S_A(1) PV_B(0) S_B(1) | PV_A(1) S_A(2) PV_B(1) S_B(2) | ...
        // so the tensor pipe works on one tile while the other tile's warpgroup does its softmax.
        // S_x(j+1) overwrites the columns P_x(j) lived in: MMAs of one thread execute in issue order
        // and P_x(j) V(j) is always issued before S_x(j+1).
        if (lane == 0) {
            uint32_t q_uses[kQBufs] = {0, 0, 0};
            uint32_t kv_base = 0;                 // key/value tiles consumed by earlier items
            uint32_t p_count[2] = {0, 0};         // P tiles consumed so far, per query tile slot
            bool ok = true;
            uint32_t n_done = 0;
            for (long long item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++n_done) {
                const Item it = decode_item(item, p);
                const int qbuf[2] = {(n_done & 1) ? 2 : 0, 1};
                const int steps[2] = {it.na, it.nb};
                // S_x(j) = Q_x K_j^T, then the barriers that fire when it (and all before it) is done
                auto issue_s = [&](int x, int j) {
                    const uint32_t kc = kv_base + j, st = kc % kKvStages;
                    ok = ok && mbar_wait(bar(B_KFULL + st), (kc / kKvStages) & 1, abort_flag, p.dev_status);
                    if (ok && j == 0) {
                        ok = mbar_wait(bar(B_QFULL + qbuf[x]), q_uses[qbuf[x]] & 1, abort_flag, p.dev_status);
                        ++q_uses[qbuf[x]];
                    }
                    if (!ok) return;
                    tc_fence_after();
                    const uint32_t q0 = sQ + qbuf[x] * TILE_BYTES, k0 = sK + st * TILE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
                        mma_bf16(tmem + COL_S0 + x * BN, make_desc(q0 + off, 16, 1024), make_desc(k0 + off, 16, 1024), IDESC_S,
                                 kk > 0 ? 1u : 0u);
                    }
                    mma_commit(bar(B_SFULL + x));
                    if (j == steps[x] - 1) mma_commit(bar(B_QEMPTY + qbuf[x]));  // last use of this Q tile
                    // K_j is free after its last reader: tile B while it still runs, else tile A
                    if (x == 1 || j >= it.nb) mma_commit(bar(B_KEMPTY + st));
                };
                // O_x (+)= P_x(j) V_j
                auto issue_pv = [&](int x, int j) {
                    const uint32_t kc = kv_base + j, st = kc % kKvStages;
                    ok = ok && mbar_wait(bar(B_P0FULL + x), p_count[x] & 1, abort_flag, p.dev_status);
                    // V_j has landed: a softmax thread waited for it before the last arrival on P0FULL
                    if (!ok) return;
                    tc_fence_after();
                    const uint32_t v0 = sV + st * TILE_BYTES;
                    // A = P from tensor memory: 16 kv columns = 8 packed 32-bit columns;
                    // B = V, MN-major: 16 kv rows = 2048 bytes; next 64 head dims one box further
                    auto pv = [&](int kk) {
                        mma_bf16_ts(tmem + COL_O0 + x * HD, tmem + COL_S0 + x * BN + kk * 8, make_desc(v0 + kk * 2048, kBoxBytes, 1024),
                                    IDESC_O, (j > 0 || kk > 0) ? 1u : 0u);
                    };
                    // the first three quarters of P arrive early: their share of the product runs while
                    // the softmax warps still work on the last quarter
#pragma unroll
                    for (int kk = 0; kk < kEarlyChunks * 2; ++kk) pv(kk);
                    ok = mbar_wait(bar(B_P1FULL + x), p_count[x] & 1, abort_flag, p.dev_status);
                    if (!ok) return;
                    ++p_count[x];
                    tc_fence_after();
#pragma unroll
                    for (int kk = kEarlyChunks * 2; kk < BN / 16; ++kk) pv(kk);
                    // V_j is free after its last reader (tile B while it still runs, else tile A) - except the
                    // last V tile of each query tile: its stage stages that tile's output first and is
                    // released by the epilogue
                    if ((x == 1 || j >= it.nb) && j != steps[x] - 1) mma_commit(bar(B_VEMPTY + st));
                    if (j == steps[x] - 1) mma_commit(bar(B_OFULL + x));
                };
                issue_s(0, 0);
                if (it.nb > 0) issue_s(1, 0);
                for (int j = 0; ok && j < it.na; ++j) {
                    issue_pv(0, j);
                    if (j + 1 < it.na) issue_s(0, j + 1);
                    if (j < it.nb) {
                        issue_pv(1, j);
                        if (j + 1 < it.nb) issue_s(1, j + 1);
                    }
                }
                kv_base += it.na;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: thread = query row
        const int x = warp >> 2;                           // 0: tile A (warps 0-3), 1: tile B (warps 4-7)
        const int wq = warp & 3;                           // TMEM lane quarter this warp may access
        const int row = wq * 32 + lane;                    // TMEM lane = query row within the tile
        const uint32_t lane_base = tmem + ((uint32_t)(wq * 32) << 16);
        const uint32_t s_addr = lane_base + COL_S0 + x * BN;
        const uint32_t o_addr = lane_base + COL_O0 + x * HD;
        uint32_t s_count = 0, o_count = 0;                 // S tiles / O tiles consumed so far by this thread
        uint32_t kv_base = 0;                              // key/value tiles consumed by earlier items
        bool ok = true;
        for (long long item = blockIdx.x; ok && item < p.n_items; item += gridDim.x) {
            const Item it = decode_item(item, p);
            const int qt = x ? it.qb : it.qa, n_kv = x ? it.nb : it.na;
            const uint32_t stage_o = (kv_base + n_kv - 1) % kKvStages;  // stage of this tile's last V tile
            const uint32_t kv0 = kv_base;                  // index of the item's first K/V tile in the rings
            kv_base += it.na;
            if (n_kv == 0) continue;                       // single-tile item: warpgroup B has nothing to do
            float m_ref = kNegInf, l = 0.f;
            for (int j = 0; j < n_kv; ++j, ++s_count) {
                const bool diag = (j == qt);
                ok = mbar_wait(bar(B_SFULL + x), s_count & 1, abort_flag, p.dev_status);  // S_j ready; O settled
                if (!ok) break;
                tc_fence_after();
                // On the diagonal tile the rows of warp w (32w .. 32w+31) see nothing right of column
                // 32w+31: only column chunks 0..w are loaded and exponentiated, chunk w with a per-row mask.
                const int nch = diag ? wq + 1 : BN / 32;
                uint32_t sr[BN];
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c < nch) tmem_ld32_issue(s_addr + c * 32, sr + c * 32);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c < nch) tmem_ld_fence32(sr + c * 32);
                if (diag) {  // masked scores become -inf: they drop out of the maximum and exponentiate to 0
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c)
                        if (c == wq) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (i > lane) sr[c * 32 + i] = __float_as_uint(kNegInf);
                        }
                }
                float mx4[4] = {kNegInf, kNegInf, kNegInf, kNegInf};  // independent chains: the maximum is latency-bound
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c < nch) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                mx4[u] = fmax3(mx4[u], __uint_as_float(sr[c * 32 + i + 2 * u]), __uint_as_float(sr[c * 32 + i + 2 * u + 1]));
                        }
                    }
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                mx *= p.scale_log2;
                float factor = 1.f;
                const bool grow_ref = mx > m_ref + kRescaleThreshold;  // first tile: m_ref = -inf
                if (grow_ref) {
                    factor = (m_ref == kNegInf) ? 0.f : ex2(m_ref - mx);
                    m_ref = mx;
                }
                if (j > 0) {
                    if (__any_sync(0xffffffffu, grow_ref)) {
#pragma unroll 1
                        for (int c0 = 0; c0 < HD; c0 += 32) {
                            float o[32];
                            tmem_ld32(o_addr + c0, o);
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= factor;
                            tmem_st32(o_addr + c0, o);
                        }
                    }
                    l *= factor;
                }
                // P = 2^(s*scale - m_ref) as bf16 pairs over the S columns (chunk c of P lands in columns
                // 16c .. 16c+15; every S column is already in registers).  The row sum is taken in fp32
                // before the rounding: the rounding errors of the 128 terms average out in the normaliser.
                const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(-m_ref, -m_ref);
                uint64_t l2a = pack2(0.f, 0.f), l2b = l2a;
#pragma unroll
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t packed[16];
                    if (c < nch) {
                        // three passes over the chunk, in place, so that 32 independent exponentials are in flight
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            float x0, x1;
                            unpack2(ffma2(pack2(__uint_as_float(sr[c * 32 + i]), __uint_as_float(sr[c * 32 + i + 1])), sc2, nm2), x0, x1);
                            sr[c * 32 + i] = __float_as_uint(x0);
                            sr[c * 32 + i + 1] = __float_as_uint(x1);
                        }
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            sr[c * 32 + i] = __float_as_uint(ex2(__uint_as_float(sr[c * 32 + i])));
                            sr[c * 32 + i + 1] = __float_as_uint(ex2(__uint_as_float(sr[c * 32 + i + 1])));
                        }
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            const float p0 = __uint_as_float(sr[c * 32 + i]), p1 = __uint_as_float(sr[c * 32 + i + 1]);
                            const float p2 = __uint_as_float(sr[c * 32 + i + 2]), p3 = __uint_as_float(sr[c * 32 + i + 3]);
                            l2a = fadd2(l2a, pack2(p0, p1));
                            l2b = fadd2(l2b, pack2(p2, p3));
                            __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), pb = __floats2bfloat162_rn(p2, p3);
                            packed[(i >> 1)] = *reinterpret_cast<uint32_t*>(&pa);
                            packed[(i >> 1) + 1] = *reinterpret_cast<uint32_t*>(&pb);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) packed[i] = 0u;
                    }
                    tmem_st16p(s_addr + c * 16, packed);
                    if (c == kEarlyChunks - 1) {  // columns 0..95 of P are in place: let their share of P V start
                        tmem_wait_st();
                        tc_fence_before();
                        // one thread also vouches for V_j: P0FULL then implies "V_j has landed", and the MMA
                        // thread, whose every barrier round trip leaves the tensor pipe dry, need not ask
                        if (wq == 0 && lane == 0) {
                            const uint32_t kc = kv0 + j;
                            ok = mbar_wait(bar(B_VFULL + kc % kKvStages), (kc / kKvStages) & 1, abort_flag, p.dev_status);
                        }
                        mbar_arrive(bar(B_P0FULL + x));
                    }
                }
                {
                    float a0, a1, b0, b1;
                    unpack2(l2a, a0, a1);
                    unpack2(l2b, b0, b1);
                    l += (a0 + a1) + (b0 + b1);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(B_P1FULL + x));
            }
            // From here to the named barrier below no thread leaves early: a thread whose wait ran out (ok ==
            // false; later waits then give up soon, the abort flag being up) still stages its row and meets the others, and the
            // barrier tells all 128 whether any of them failed, so that they give up at the same item.
            if (ok) ok = mbar_wait(bar(B_OFULL + x), o_count & 1, abort_flag, p.dev_status);
            ++o_count;
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            // O row -> bf16 -> the shared-memory stage that held this tile's last V tile (every MMA that
            // read it is done), in the 128-byte-swizzled box layout, then one TMA store per box; rows
            // past T are dropped by the store.  The stage goes back to the producer once read.
            const uint32_t stage = sV + stage_o * TILE_BYTES + row * 128;
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 64) {
                uint32_t o[64];
                tmem_ld32_issue(o_addr + c0, o);
                tmem_ld32_issue(o_addr + c0 + 32, o + 32);
                tmem_wait_ld();
                tmem_ld_fence32(o);
                tmem_ld_fence32(o + 32);
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(o[q8 * 8 + i]) * inv;
                    const uint4 w = pack8(f);
                    const uint32_t dst = stage + (c0 >> 6) * kBoxBytes + ((q8 ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
                }
            }
            tc_fence_before();
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            uint32_t any_failed;  // the warpgroup's 128 rows are staged; did a wait run out in any of its threads?
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %2, 0;\n\t"
                "bar.red.or.pred p, %1, 128, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(any_failed)
                : "r"(1 + x), "r"(ok ? 0u : 1u)
                : "memory");
            if (any_failed) break;
            if (wq == 0 && lane == 0) {
                for (int bx = 0; bx < NB; ++bx)
                    tma_store_3d(&mapO, sV + stage_o * TILE_BYTES + bx * kBoxBytes, bx * 64, qt * BM, it.bh);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_arrive(bar(B_VEMPTY + stage_o));
            }
            // the next item's first P V overwrites O: it is issued only after this thread's next
            // arrival on P0FULL, which follows these loads in program order
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // this thread's stores have landed
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---- host side
// [slabs][rows][hd] bf16 with `stride_rows` rows between slabs; box = 64 x 128 x 1, 128-byte swizzle,
// rows past `rows` read as zeros.
static bool make_map(CUtensorMap* m, const void* ptr, int hd, int rows, long long stride_rows, long long slabs)
{
    return make_slab_map(m, ptr, hd, rows, stride_rows, slabs, 128);
}

static int gcd_int(int a, int b)
{
    while (b) {
        int t = a % b;
        a = b;
        b = t;
    }
    return a;
}

template <int HD>
static cudaError_t launch_t(const PrefillArgs& a, uint32_t* dev_status, cudaStream_t stream)
{
    static PerDeviceOnce limit_raised;
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    e = raise_smem_limit_once(limit_raised, dev, block_prefill_tc_kernel<HD>, smem_bytes<HD>());
    if (e != cudaSuccess) return e;
    const long long slabs = (long long)a.B * a.H;
    CUtensorMap mq, mk, mv, mo;
    if (!make_map(&mq, a.q, HD, a.T, a.T, slabs) || !make_map(&mk, a.k, HD, a.T, a.kv_seq_stride, slabs) ||
        !make_map(&mv, a.v, HD, a.T, a.kv_seq_stride, slabs) || !make_map(&mo, a.out, HD, a.T, a.T, slabs))
        return cudaErrorInvalidValue;
    Params p;
    p.dev_status = dev_status;
    p.T = a.T;
    p.n_qtiles = (a.T + BM - 1) / BM;
    p.n_classes = (p.n_qtiles + 1) / 2;
    p.n_items = slabs * p.n_classes;
    p.scale_log2 = a.scale_log2;
    // one persistent CTA per SM; a grid size coprime to the number of classes makes every CTA
    // cycle through all classes (heavy and light items alike)
    long long grid = p.n_items < sms ? p.n_items : sms;
    while (grid > 1 && p.n_items > grid && gcd_int((int)grid, p.n_classes) != 1) --grid;
    return launch_pdl(block_prefill_tc_kernel<HD>, dim3((unsigned)grid), dim3(kThreads), (size_t)smem_bytes<HD>(), stream, mq, mk, mv, mo, p);
}

}  // namespace pf

bool prefill_tc_supported(const PrefillArgs& a)
{
    auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return (a.hd == 64 || a.hd == 128) && al(a.q) && al(a.k) && al(a.v) && al(a.out) && tensor_map_encode_fn() != nullptr;
}

cudaError_t launch_block_prefill_tc(const PrefillArgs& a, uint32_t* dev_status, cudaStream_t stream)
{
    return a.hd == 64 ? pf::launch_t<64>(a, dev_status, stream) : pf::launch_t<128>(a, dev_status, stream);
}

}  // namespace bt
