// Block-decoder prefill attention on the 5th-generation tensor cores (paper sections 2.1, 2.3:
// the prefill stage processes all prompt blocks in parallel; causal over blocks).
//
// Persistent kernel, one CTA per SM (all of its shared memory and its 512 tensor-memory columns).
// A work item is a pair of neighbouring 128-row query tiles of one (sequence, head); the two tiles
// walk the same 64-row key/value tiles 0 .. diagonal, so K and V are loaded once for both.  Each query
// tile owns TWO score buffers in tensor memory (2 x 64 fp32 columns): S(j+1) and S(j+2) are computed
// while the softmax warps still work on S(j), so those warps never wait for the tensor pipe and the
// pipe never waits for more than the P tile it is about to multiply.  Roles:
//   warps 0-3 / 4-7 : softmax of query tile A / B - each thread owns one query row (= one TMEM lane)
//                     and holds its 64 scores in registers: one batch of tensor-memory loads, row
//                     maximum, exp2 (packed fp32x2 multiply-adds around it), bf16 P written over the S
//                     columns, running row sum; on the two diagonal tiles a warp skips the column
//                     chunks that are masked for all of its rows.  O is rescaled in TMEM only when the
//                     row maximum grew by more than 2^8 (otherwise the old reference is kept, exact
//                     because O and the row sum share it), after the previous P V has completed.  At
//                     the end of an item the rows go through shared memory (the tile's own, by then
//                     dead, Q buffer) to a TMA store.
//   warp 8 (1 lane) : TMA producer - Q tiles (Q_A double-buffered an item ahead), K and V rings of
//                     four 64-row stages, 128-byte swizzle
//   warps 9, 10     : tcgen05.mma issuers of tile A and tile B (the whole warp walks the loop, an elected lane issues) -
//                     S = Q K^T into tensor memory, O += P V with P read from tensor memory (the
//                     probabilities never visit shared memory), each in the order PV(j) S(j+2)
// All waits are bounded in wall time: one that runs out raises BT_DEV_TIMEOUT and the CTA winds down.
#include <cuda.h>

#include <memory>
#include <mutex>
#include <utility>
#include <vector>

#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"
#include "bt_tcgen05.cuh"
#include "bt_tensor_map.h"

namespace bt {
namespace pf {

constexpr int BM = 128;             // query rows per tile
constexpr int BN = 64;              // key/value rows per tile
constexpr int kQBoxBytes = BM * 128;   // one TMA box of Q or O: 128 rows x 64 bf16 (128 bytes, swizzled)
constexpr int kKvBoxBytes = BN * 128;  // one TMA box of K or V: 64 rows x 64 bf16
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

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed fp32 pairs (one instruction for two lanes' worth of work on sm_100).
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
// query tile t needs the 64-row key/value tiles 0 .. 2t+1.  An item is a pair of neighbouring query
// tiles taken from the top: class k holds tiles A = n-1-2k (na = 2A+2 tile steps) and B = A-1
// (nb = na-2 steps; absent when A is tile 0).  The two tiles of an item walk the same key/value
// tiles, so K and V are loaded once for both and their work is nearly equal, which keeps both softmax
// warpgroups busy.  Items are numbered item = bh * m + k (m = ceil(n/2) classes) and CTA c processes
// items c, c+G, c+2G, ... with the grid size G coprime to m, so every CTA cycles through all classes
// (balanced work) while the classes of one (sequence, head) run at the same time on neighbouring
// CTAs and share its K and V through L2.
struct Params {
    uint32_t* dev_status;
    int T, n_qtiles, n_classes;
    long long n_items;
    float scale_log2;
};

// warps 0-3: softmax warpgroup of tile A, warps 4-7: of tile B
constexpr int kProducerWarp = 8, kMmaWarp = 9;  // warp 9 issues for tile A, warp 10 for tile B
constexpr int kThreads = 352;
constexpr int kQBufs = 3;                   // Q_A alternates between buffers 0 and 2, Q_B lives in buffer 1
constexpr int kKvStages = 4;
__device__ __forceinline__ int qbuf_a(uint32_t n_done) { return (n_done & 1) ? 2 : 0; }
__device__ __forceinline__ int qbuf_b(uint32_t) { return 1; }

// Which items a CTA processes, in which order.  Small launches (the usual case) carry a table made on the host:
// items dealt heaviest first to the least loaded CTA, inside waves of (sequence, head) slabs whose K and V fit
// the L2 together - item costs differ eightfold at a long prompt, and a plain round robin leaves the slowest
// CTA 10 % above the mean.  Larger launches use item = c, c + G, c + 2G, ... (enough items per CTA to even out).
constexpr int kMaxTableCtas = 192, kMaxTableItems = 4096;
struct Schedule {
    int use_table;
    uint16_t start[kMaxTableCtas + 1];   // CTA c owns order[start[c] .. start[c+1])
    uint16_t order[kMaxTableItems];
};

// barrier slots in shared memory
enum {
    B_QFULL = 0,                       // [kQBufs]  TMA -> MMA
    B_QEMPTY = B_QFULL + kQBufs,       // [kQBufs]  epilogue (output staged in the buffer has been read by its store) -> TMA
    B_KFULL = B_QEMPTY + kQBufs,       // [kKvStages]  K_j and V_j of a stage have both landed
    B_KEMPTY = B_KFULL + kKvStages,    // [kKvStages]  both tiles' P V products on the stage are done (two arrivals)
    B_SFULL = B_KEMPTY + kKvStages,    // [2 tiles][2 buffers]: S ready
    B_PFULL = B_SFULL + 4,             // [2 tiles][2 buffers]: 128 softmax threads have written P over it
    B_PVDONE = B_PFULL + 4,            // [2 tiles]: one completion per P V product (O may be rescaled after it)
    B_OFULL = B_PVDONE + 2,            // [2 tiles]: last P V of the item done
    B_COUNT = B_OFULL + 2
};

template <int HD>
constexpr int smem_bytes()
{
    // Q tiles (HD/64 boxes of 16 KB), K and V stages (HD/64 boxes of 8 KB), barriers, plus 1024 to align
    return 1024 + (HD / 64) * (kQBoxBytes * kQBufs + kKvBoxBytes * 2 * kKvStages) + 512;
}

constexpr uint32_t kTmemCols = 512;  // S_A0, S_A1, S_B0, S_B1 (64 columns each), O_A, O_B (head_dim columns each)

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
    it.na = 2 * it.qa + 2;
    it.nb = 2 * it.qb + 2;  // 0 when qb == -1
    return it;
}

// Position i of this CTA's walk over its items.
__device__ __forceinline__ long long walk_begin(const Schedule& sc) { return sc.use_table ? sc.start[blockIdx.x] : blockIdx.x; }
__device__ __forceinline__ bool walk_done(const Schedule& sc, const Params& p, long long i)
{
    return sc.use_table ? i >= sc.start[blockIdx.x + 1] : i >= p.n_items;
}
__device__ __forceinline__ long long walk_next(const Schedule& sc, long long i) { return sc.use_table ? i + 1 : i + gridDim.x; }
__device__ __forceinline__ long long walk_item(const Schedule& sc, long long i) { return sc.use_table ? sc.order[i] : i; }

template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
block_prefill_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO, Params p,
                        const __grid_constant__ Schedule sched)
{
    constexpr int NB = HD / 64;                 // TMA boxes per operand tile
    constexpr uint32_t Q_TILE_BYTES = NB * kQBoxBytes, KV_TILE_BYTES = NB * kKvBoxBytes;
    constexpr uint32_t IDESC_S = make_idesc(BM, BN, false);
    constexpr uint32_t IDESC_O = make_idesc(BM, HD, true);
    // TMEM columns: S (fp32) / P (bf16 pairs, in place), two buffers for each of tiles A and B, then O of A and B
    constexpr uint32_t COL_S0 = 0, COL_O0 = 4 * BN;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sQ = base;                               // kQBufs tiles
    const uint32_t sK = sQ + kQBufs * Q_TILE_BYTES;         // kKvStages tiles
    const uint32_t sV = sK + kKvStages * KV_TILE_BYTES;     // kKvStages tiles
    const uint32_t sBar = sV + kKvStages * KV_TILE_BYTES;   // B_COUNT x 8 bytes
    uint8_t* gen_tail = gen_base + (sBar - base);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_tail + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_tail + B_COUNT * 8 + 8);
    auto bar = [&](int i) { return sBar + 8u * i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(bar(i), (i >= B_PFULL && i < B_PFULL + 4) ? 128u : (i >= B_KEMPTY && i < B_KEMPTY + kKvStages) ? 2u : 1u);
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
    if (warp == kProducerWarp && lane == 0 && !walk_done(sched, p, walk_begin(sched))) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapQ) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
        const Item it = decode_item(walk_item(sched, walk_begin(sched)), p);
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
            uint32_t q_uses[4] = {0, 0, 0, 0};
            uint32_t kv_count = 0;   // key/value tiles loaded so far (K and V advance together)
            uint32_t n_done = 0;     // items processed by this CTA
            bool ok = true;
            for (long long wi = walk_begin(sched); ok && !walk_done(sched, p, wi); wi = walk_next(sched, wi), ++n_done) {
                const long long item = walk_item(sched, wi);
                const Item it = decode_item(item, p);
                auto load_q = [&](int buf, int qt) {
                    ok = ok && mbar_wait(bar(B_QEMPTY + buf), (q_uses[buf] & 1) ^ 1, abort_flag, p.dev_status);
                    if (!ok) return;
                    ++q_uses[buf];
                    mbar_expect_tx(bar(B_QFULL + buf), Q_TILE_BYTES);
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sQ + buf * Q_TILE_BYTES + bx * kQBoxBytes, &mapQ, bar(B_QFULL + buf), bx * 64, qt * BM, it.bh);
                };
                auto load_kv = [&](int j) {
                    const uint32_t st = kv_count % kKvStages, par = ((kv_count / kKvStages) & 1) ^ 1;
                    ok = ok && mbar_wait(bar(B_KEMPTY + st), par, abort_flag, p.dev_status);
                    if (!ok) return;
                    mbar_expect_tx(bar(B_KFULL + st), 2 * KV_TILE_BYTES);  // K and V of a stage arrive on one barrier
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sK + st * KV_TILE_BYTES + bx * kKvBoxBytes, &mapK, bar(B_KFULL + st), bx * 64, j * BN, it.bh);
                    for (int bx = 0; bx < NB; ++bx)
                        tma_load_3d(sV + st * KV_TILE_BYTES + bx * kKvBoxBytes, &mapV, bar(B_KFULL + st), bx * 64, j * BN, it.bh);
                    ++kv_count;
                };
                // Q_A and the first two key/value tiles come first (tile A's first two products need just these);
                // Q_B, whose buffer may be handed back late by the previous item's epilogue, must not hold them up
                load_q(qbuf_a(n_done), it.qa);
                load_kv(0);
                load_kv(1);
                if (it.nb > 0) load_q(qbuf_b(n_done), it.qb);
                for (int j = 2; ok && j < it.na; ++j) load_kv(j);
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // ------------------------------------------------------------------ MMA issuers, one warp per query tile
        // Issue order of tile x:  S_x(0) S_x(1) | PV_x(0) S_x(2) | PV_x(1) S_x(3) | ...
        // S_x(j) goes to score buffer j & 1 of the tile; S_x(j+2) overwrites the columns P_x(j) lived in: the
        // instructions of one thread execute in issue order and P_x(j) V(j) is issued before S_x(j+2).  The two
        // warps do not order their work against each other; the tensor pipe takes the instructions as they come.
        // A key/value stage is handed back by two arrivals, one per tile (tile A arrives twice for the tiles that
        // only it reads).  The whole warp walks the loop - control flow stays warp-uniform, every wait's outcome
        // is agreed on by a vote - and one elected lane issues: a lone lane inside a divergent branch issues
        // tcgen05.mma slower than the tensor pipe runs them.
        {
            const int x = warp - kMmaWarp;
            auto wait_all = [&](uint32_t b, uint32_t parity) {
                const bool r = mbar_wait(b, parity, abort_flag, p.dev_status);
                return __all_sync(0xffffffffu, r) != 0;
            };
            uint32_t q_uses[4] = {0, 0, 0, 0};
            uint32_t kv_base = 0;                 // key/value tiles consumed by earlier items
            uint32_t p_count = 0;                 // P tiles consumed so far
            bool ok = true;
            uint32_t n_done = 0;
            for (long long wi = walk_begin(sched); ok && !walk_done(sched, p, wi); wi = walk_next(sched, wi), ++n_done) {
                const long long item = walk_item(sched, wi);
                const Item it = decode_item(item, p);
                const int qbuf = x ? qbuf_b(n_done) : qbuf_a(n_done);
                const int steps = x ? it.nb : it.na;
                // S_x(j) = Q_x K_j^T, then the barriers that fire when it (and all before it) is done
                auto issue_s = [&](int j) {
                    const uint32_t kc = kv_base + j, st = kc % kKvStages;
                    ok = ok && wait_all(bar(B_KFULL + st), (kc / kKvStages) & 1);
                    if (ok && j == 0) {
                        ok = wait_all(bar(B_QFULL + qbuf), q_uses[qbuf] & 1);
                        ++q_uses[qbuf];
                    }
                    if (!ok) return;
                    tc_fence_after();
                    // Descriptor low words: the tile's address in 16-byte units plus the leading-dimension field -
                    // one add per operand and instruction.  16 head dims = 32 bytes inside a swizzled 128-byte row;
                    // the next 64 head dims are one box further.
                    const uint32_t qlo = ((sQ + qbuf * Q_TILE_BYTES) >> 4) | (1u << 16);
                    const uint32_t klo = ((sK + st * KV_TILE_BYTES) >> 4) | (1u << 16);
                    const uint32_t d_s = tmem + COL_S0 + (uint32_t)(x * 2 + (j & 1)) * BN;
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < HD / 16; ++kk) {
                            const uint32_t qoff = (uint32_t)(((kk >> 2) * kQBoxBytes + (kk & 3) * 32) >> 4);
                            const uint32_t koff = (uint32_t)(((kk >> 2) * kKvBoxBytes + (kk & 3) * 32) >> 4);
                            mma_bf16(d_s, desc_words(qlo + qoff, kDescHiSw128), desc_words(klo + koff, kDescHiSw128), IDESC_S, kk > 0 ? 1u : 0u);
                        }
                        mma_commit(bar(B_SFULL + x * 2 + (j & 1)));
                    }
                    __syncwarp();
                };
                // O_x (+)= P_x(j) V_j
                auto issue_pv = [&](int j) {
                    const uint32_t kc = kv_base + j, st = kc % kKvStages;
                    ok = ok && wait_all(bar(B_PFULL + x * 2 + (p_count & 1)), (p_count >> 1) & 1);
                    if (!ok) return;
                    ++p_count;
                    tc_fence_after();
                    // A = P from tensor memory: 16 kv columns = 8 packed 32-bit columns;
                    // B = V, MN-major: 16 kv rows = 2048 bytes; the next 64 head dims are one box further
                    const uint32_t vlo = ((sV + st * KV_TILE_BYTES) >> 4) | ((uint32_t)(kKvBoxBytes >> 4) << 16);
                    const uint32_t a_p = tmem + COL_S0 + (uint32_t)(x * 2 + (j & 1)) * BN;
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < BN / 16; ++kk)
                            mma_bf16_ts(tmem + COL_O0 + x * HD, a_p + kk * 8, desc_words(vlo + (uint32_t)kk * 128u, kDescHiSw128), IDESC_O,
                                        (j > 0 || kk > 0) ? 1u : 0u);
                        mma_commit(bar(B_PVDONE + x));
                        // the stage (K_j and V_j) is free after its last reader
                        mma_commit(bar(B_KEMPTY + st));
                        if (x == 0 && j >= it.nb) mma_commit(bar(B_KEMPTY + st));  // tile B does not read this one
                        if (j == steps - 1) mma_commit(bar(B_OFULL + x));
                    }
                    __syncwarp();
                };
                if (steps > 0) {
                    issue_s(0);
                    issue_s(1);
                    for (int j = 0; ok && j < steps; ++j) {
                        issue_pv(j);
                        if (j + 2 < steps) issue_s(j + 2);
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
        const uint32_t o_addr = lane_base + COL_O0 + x * HD;
        uint32_t s_count = 0, o_count = 0;                 // S tiles / O tiles consumed so far by this thread
        uint32_t n_done = 0;
        bool ok = true;
        for (long long wi = walk_begin(sched); ok && !walk_done(sched, p, wi); wi = walk_next(sched, wi), ++n_done) {
            const long long item = walk_item(sched, wi);
            const Item it = decode_item(item, p);
            const int qt = x ? it.qb : it.qa, n_kv = x ? it.nb : it.na;
            const int qbuf = x ? qbuf_b(n_done) : qbuf_a(n_done);
            if (n_kv == 0) continue;                       // single-tile item: warpgroup B has nothing to do
            float m_ref = kNegInf, l = 0.f;
            for (int j = 0; j < n_kv; ++j, ++s_count) {
                const uint32_t buf = s_count & 1;          // = j & 1: every tile takes an even number of steps
                const uint32_t s_addr = lane_base + COL_S0 + (uint32_t)(x * 2 + buf) * BN;
                ok = mbar_wait(bar(B_SFULL + x * 2 + buf), (s_count >> 1) & 1, abort_flag, p.dev_status);
                if (!ok) break;
                tc_fence_after();
                // The last two key/value tiles straddle the diagonal.  Row r of the query tile sees column c of
                // tile j iff c <= r - 64 (j - 2 qt); of a warp's rows 32 wq .. 32 wq + 31 the 32-column chunk
                // `part` = wq - 2 (j - 2 qt) is masked per row, the chunks before it are fully visible and the
                // chunks after it are masked for all of its rows and are neither loaded nor exponentiated.
                const int dj = j - 2 * qt;                 // 0 or 1 on the diagonal tiles, negative before them
                const int part = dj >= 0 ? wq - 2 * dj : BN / 32;
                const int nch = part < 0 ? 0 : (part + 1 < BN / 32 ? part + 1 : BN / 32);
                uint32_t sr[BN];
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c < nch) tmem_ld32_issue(s_addr + c * 32, sr + c * 32);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c < nch) tmem_ld_fence32(sr + c * 32);
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if (c == part) {  // masked scores become -inf: they drop out of the maximum and exponentiate to 0
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i > lane) sr[c * 32 + i] = __float_as_uint(kNegInf);
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
                        // O still receives P(j-1) V(j-1): that product was issued when this thread's previous P tile
                        // was announced and is the (s_count - 1)-th completion on the tile's barrier.  (The product
                        // before it was complete before S(j) was announced, so the parity cannot be stale.)
                        ok = mbar_wait(bar(B_PVDONE + x), (s_count - 1) & 1, abort_flag, p.dev_status);
                        if (!__all_sync(0xffffffffu, ok)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
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
                // before the rounding: the rounding errors of the terms average out in the normaliser.
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
                }
                {
                    float a0, a1, b0, b1;
                    unpack2(l2a, a0, a1);
                    unpack2(l2b, b0, b1);
                    l += (a0 + a1) + (b0 + b1);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(B_PFULL + x * 2 + buf));
            }
            // From here to the named barrier below no thread leaves early: a thread whose wait ran out (ok ==
            // false; later waits then give up soon, the abort flag being up) still stages its row and meets the others, and the
            // barrier tells all 128 whether any of them failed, so that they give up at the same item.
            if (ok) ok = mbar_wait(bar(B_OFULL + x), o_count & 1, abort_flag, p.dev_status);
            ++o_count;
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            // O row -> bf16 -> the tile's own Q buffer (every MMA that read it is done), in the
            // 128-byte-swizzled box layout, then one TMA store per box; rows past T are dropped by the
            // store.  The buffer goes back to the producer once read.
            const uint32_t stage = sQ + qbuf * Q_TILE_BYTES + row * 128;
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
                    const uint32_t dst = stage + (c0 >> 6) * kQBoxBytes + ((q8 ^ (row & 7)) << 4);
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
                    tma_store_3d(&mapO, sQ + qbuf * Q_TILE_BYTES + bx * kQBoxBytes, bx * 64, qt * BM, it.bh);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_arrive(bar(B_QEMPTY + qbuf));
            }
            // the next item's first P V overwrites O: it is issued only after this thread's next
            // arrival on PFULL, which follows these loads in program order
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
// [slabs][rows][hd] bf16 with `stride_rows` rows between slabs; box = 64 x box_rows x 1, 128-byte swizzle,
// rows past `rows` read as zeros.
static bool make_map(CUtensorMap* m, const void* ptr, int hd, int rows, long long stride_rows, long long slabs, int box_rows)
{
    return make_slab_map(m, ptr, hd, rows, stride_rows, slabs, box_rows);
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

// The table for `slabs` (sequence, head) pairs of `n_qtiles` query tiles on `grid` CTAs; false when it does not fit.
// Cost of the class-k item: its longer tile's steps (2 (n_qtiles - 2k)) plus two for what an item pays around
// them.  Waves of `wave` slabs are dealt one after the other, each heaviest class first, every item to the CTA
// with the least work so far; a CTA's list keeps the order of dealing, so the slabs of a wave are in flight
// together and find each other's K and V in the L2.
static bool build_schedule(Schedule* sc, long long slabs, int n_qtiles, int n_classes, int grid, int hd, int T)
{
    const long long n_items = slabs * n_classes;
    if (n_items > kMaxTableItems || grid > kMaxTableCtas) return false;
    if (n_classes < 3) return false;  // two classes alternate evenly under the round robin already
    const long long kv_bytes_per_slab = 2ll * T * hd * 2;
    long long wave = (48ll << 20) / (kv_bytes_per_slab > 0 ? kv_bytes_per_slab : 1);
    const long long wave_min = 2 * ((grid + n_classes - 1) / n_classes);  // two rounds of items per wave at least
    if (wave < wave_min) wave = wave_min;
    if (wave > slabs) wave = slabs;
    std::vector<long long> load(grid, 0);
    std::vector<std::vector<uint16_t>> lists(grid);
    for (long long w0 = 0; w0 < slabs; w0 += wave) {
        const long long w1 = w0 + wave < slabs ? w0 + wave : slabs;
        for (int k = 0; k < n_classes; ++k) {
            const int cost = 2 * (n_qtiles - 2 * k) + 2;
            for (long long bh = w0; bh < w1; ++bh) {
                int best = 0;
                for (int c = 1; c < grid; ++c)
                    if (load[c] < load[best]) best = c;
                load[best] += cost;
                lists[best].push_back((uint16_t)(bh * n_classes + k));
            }
        }
    }
    sc->use_table = 1;
    int pos = 0;
    for (int c = 0; c < grid; ++c) {
        sc->start[c] = (uint16_t)pos;
        for (uint16_t it : lists[c]) sc->order[pos++] = it;
    }
    for (int c = grid; c <= kMaxTableCtas; ++c) sc->start[c] = (uint16_t)pos;
    return true;
}

// Tables are kept per shape: building one costs a few hundred microseconds.
struct ScheduleKey {
    long long slabs;
    int n_qtiles, grid, hd, T;
    bool operator==(const ScheduleKey& o) const { return slabs == o.slabs && n_qtiles == o.n_qtiles && grid == o.grid && hd == o.hd && T == o.T; }
};
static void cached_schedule(Schedule* out, long long slabs, int n_qtiles, int n_classes, int grid, int hd, int T)
{
    static std::vector<std::pair<ScheduleKey, std::unique_ptr<Schedule>>> cache;
    const ScheduleKey key{slabs, n_qtiles, grid, hd, T};
    std::lock_guard<std::mutex> lock(setup_mutex());
    for (auto& e : cache)
        if (e.first == key) {
            *out = *e.second;
            return;
        }
    std::unique_ptr<Schedule> sc(new Schedule());
    if (!build_schedule(sc.get(), slabs, n_qtiles, n_classes, grid, hd, T)) sc->use_table = 0;
    if (cache.size() >= 32) cache.erase(cache.begin());
    *out = *sc;
    cache.emplace_back(key, std::move(sc));
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
    if (!make_map(&mq, a.q, HD, a.T, a.T, slabs, BM) || !make_map(&mk, a.k, HD, a.T, a.kv_seq_stride, slabs, BN) ||
        !make_map(&mv, a.v, HD, a.T, a.kv_seq_stride, slabs, BN) || !make_map(&mo, a.out, HD, a.T, a.T, slabs, BM))
        return cudaErrorInvalidValue;
    Params p;
    p.dev_status = dev_status;
    p.T = a.T;
    p.n_qtiles = (a.T + BM - 1) / BM;
    p.n_classes = (p.n_qtiles + 1) / 2;
    p.n_items = slabs * p.n_classes;
    p.scale_log2 = a.scale_log2;
    // one persistent CTA per SM
    long long grid = p.n_items < sms ? p.n_items : sms;
    static thread_local Schedule sc;  // 8 KB: passed to the kernel by value
    cached_schedule(&sc, slabs, p.n_qtiles, p.n_classes, (int)grid, HD, a.T);
    if (!sc.use_table) {
        // no table: a grid size coprime to the number of classes makes every CTA cycle through all classes
        // (heavy and light items alike)
        while (grid > 1 && p.n_items > grid && gcd_int((int)grid, p.n_classes) != 1) --grid;
    }
    return launch_pdl(block_prefill_tc_kernel<HD>, dim3((unsigned)grid), dim3(kThreads), (size_t)smem_bytes<HD>(), stream, mq, mk, mv, mo, p, sc);
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
