// Block-decoder decode step with several queries per (sequence, head): the "densified" block decoder
// the paper proposes in its discussion of future work (a block is represented by L_B sub-block tokens
// instead of one, so a decode step appends L_B rows to the block cache and runs L_B queries, query i
// seeing every cached row and the new rows 0..i).  The cache is fetched once per block for all L_B
// queries, which is the point of the proposal.
//
// Same streaming structure as the single-query kernel: one persistent CTA per SM, eight warps, every
// warp on its own with a ring of three 8 KB shared-memory stages (4 KB of K rows + the same V rows:
// 32 rows at head_dim 64, 16 at 128) kept full across item boundaries.  What differs is the arithmetic: with m queries per row the work
// is a real [m x hd] x [hd x rows] contraction, m times the single-query flops per byte, which the
// CUDA cores cannot hide behind the stream - so the stages are filled by TMA tensor copies with the
// 128-byte swizzle (conflict-free ldmatrix) and scores and weighted sums run on the tensor cores as
// m16n8k16 warp-level MMAs, the m <= 8 queries in rows 0..7 of the 16-row tile.  (A CTA-wide
// tcgen05 tile would need 64 or 128 query rows per (sequence, head); there are at most 8.)  P is
// rounded to bf16 where it meets V, the row sum is taken in fp32 before the rounding.
//
// The new rows are stored into the cache by the warp that owns the item before it requests the
// item's first chunk (generic-proxy stores, proxy fence, then the TMA reads), so they stream through
// the ring like every other row and the causal rule among them is one comparison per score.  Lengths
// are raised through the per-sequence arrival counter exactly as in the single-query kernel.
#include <cuda.h>

#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"
#include "bt_tensor_map.h"

namespace bt {
namespace mq {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 3;
constexpr int CHUNK_BYTES = 4096;              // K rows of one chunk (and as many bytes of V rows)
constexpr int STAGE_BYTES = 2 * CHUNK_BYTES;   // K chunk, then V chunk
// A row is HD/64 TMA boxes of 64 elements (128 bytes, the swizzle span); a chunk holds box after box,
// each ROWS rows of 128 bytes.
template <int HD>
struct Geo {
    static_assert(HD == 64 || HD == 128, "head_dim must be 64 or 128");
    static constexpr int NBOX = HD / 64;
    static constexpr int ROWS = CHUNK_BYTES / (HD * 2);   // cache rows per chunk: 32 or 16
    static constexpr int BOX_BYTES = ROWS * 128;
};
constexpr int kPrefetchChunks = 16;            // chunks of a warp's first item warmed in L2 ahead of the dependent-launch wait
constexpr uint32_t kPollLimit = 1u << 24;      // polls of one wait before giving up (each poll suspends briefly)
constexpr int kSmemBytes = kWarps * kStages * STAGE_BYTES + kWarps * kStages * 8 + 1024;  // + room to align to 1 KB

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) { return mbar_wait_polls(bar, parity, kPollLimit); }

// one box (64 elements from column `col` x ROWS rows of one slab) global -> shared, completion counted on
// the mbarrier
__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, uint32_t bar, int col, int row, int slab)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(col), "r"(row), "r"(slab), "r"(bar)
        : "memory");
}

// four 8x8 bf16 matrices, one 16-byte row per lane address; .trans hands each lane a column pair
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// D (16x8 fp32) += A (16x16 bf16, rows 8..15 zero) x B (16x8 bf16)
__device__ __forceinline__ void mma_rows0to7(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct Work {
    int bh, b, n0, n, nchunks;
    bool append, overflow;
};
template <int ROWS>
__device__ __forceinline__ Work decode_work(int item, const MultiDecodeArgs& a)
{
    Work w;
    w.bh = item;
    w.b = item / a.H;
    int n0 = a.len[w.b];
    n0 = n0 < 0 ? 0 : (n0 > a.n_max ? a.n_max : n0);
    w.n0 = n0;
    w.append = n0 + a.m <= a.n_max;   // all m rows or none: a sequence without room is flagged and attended as it is
    w.overflow = !w.append;
    w.n = w.append ? n0 + a.m : n0;
    w.nchunks = (w.n + ROWS - 1) / ROWS;
    return w;
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
block_decode_mq_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, MultiDecodeArgs a)
{
    using G = Geo<HD>;
    constexpr int ROWS = G::ROWS, NBOX = G::NBOX, BOX_BYTES = G::BOX_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // the swizzle pattern repeats every 1 KB
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring0 = base + warp * (kStages * STAGE_BYTES);
    const uint32_t bar0 = base + kWarps * kStages * STAGE_BYTES + warp * (kStages * 8);

    if (lane == 0) {
        for (int s = 0; s < kStages; ++s)
            mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
    }
    __syncwarp();
    pdl_launch_dependents();

    const int n_items = a.B * a.H;
    const int stride = kWarps * gridDim.x;
    const int first = warp * gridDim.x + blockIdx.x;   // neighbouring items go to different SMs
    bf16* Kall = reinterpret_cast<bf16*>(a.k);
    bf16* Vall = reinterpret_cast<bf16*>(a.v);
    // While the kernel before this one drains, warm L2 with the start of this warp's first item (CTAs
    // placed early sit idle until the previous kernel's last CTA is gone, and HBM is not busy in that
    // tail).  A prefetch returns nothing to the thread, so it is safe ahead of the wait; the row count
    // comes from a look at the length that may be out of date (read past L1) and is only a hint.
    if (first < n_items) {
        int n_hint = __ldcg(a.len + first / a.H);
        n_hint = n_hint < 0 ? 0 : (n_hint > a.n_max ? a.n_max : n_hint);
        const size_t off = (size_t)first * a.n_max * HD;
        const int lines = (min(kPrefetchChunks * CHUNK_BYTES, n_hint * HD * 2) + 127) / 128;
        for (int i = lane; i < lines; i += 32) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Kall + off) + (size_t)i * 128));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Vall + off) + (size_t)i * 128));
        }
    }
    pdl_wait();  // nothing above wrote global memory, or used a value read from it for more than a prefetch hint
    const bf16* Knew = reinterpret_cast<const bf16*>(a.k_new);
    const bf16* Vnew = reinterpret_cast<const bf16*>(a.v_new);

    // ---- producer cursor (kept by every lane, acted on by lane 0): next chunk to request
    int p_item = first, p_c = 0;
    Work pw = {};
    auto p_seek = [&]() {  // move to the next item that has rows; its new rows go into the cache first
        while (p_item < n_items) {
            pw = decode_work<ROWS>(p_item, a);
            if (pw.append) {
                for (int i = lane; i < a.m * (HD / 8); i += 32) {   // 16-byte pieces of the m new K rows and V rows
                    const size_t src = ((size_t)pw.bh * a.m) * HD + (size_t)i * 8;
                    const size_t dst = ((size_t)pw.bh * a.n_max + pw.n0) * HD + (size_t)i * 8;
                    *reinterpret_cast<uint4*>(Kall + dst) = ld_plain(Knew + src);
                    *reinterpret_cast<uint4*>(Vall + dst) = ld_plain(Vnew + src);
                }
                // the copy engine reads these rows next: order the stores before its reads
                asm volatile("fence.proxy.async;" ::: "memory");
                __syncwarp();
            }
            if (pw.nchunks > 0) {
                p_c = 0;
                return;
            }
            p_item += stride;
        }
    };
    uint32_t issued = 0, consumed = 0;
    auto issue_one = [&]() {
        if (p_item >= n_items) return;
        const uint32_t st = issued % kStages;
        if (lane == 0) {
            const uint32_t bar = bar0 + 8 * st, dst = ring0 + st * STAGE_BYTES;
            // a box is always delivered whole (rows past the slab arrive as zeros)
            mbar_expect_tx(bar, (uint32_t)STAGE_BYTES);
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx) {
                tma_load_box(dst + bx * BOX_BYTES, &mapK, bar, bx * 64, p_c * ROWS, pw.bh);
                tma_load_box(dst + CHUNK_BYTES + bx * BOX_BYTES, &mapV, bar, bx * 64, p_c * ROWS, pw.bh);
            }
        }
        ++issued;
        if (++p_c == pw.nchunks) {
            p_item += stride;
            p_seek();
        }
    };
    p_seek();
    for (int s = 0; s < kStages; ++s) issue_one();

    // ---- consumer.  Lane (g, t) = (lane / 4, lane % 4) owns query row g and, of every 8 columns, 2t and 2t+1.
    const int g = lane >> 2, t = lane & 3;
    // Lane-constant parts of the ldmatrix addresses.  16-byte piece p of row r of a chunk lies in box p / 8
    // at r * 128 + ((p % 8) ^ (r % 8)) * 16.  K: one instruction reads 8 rows x the four pieces 4h..4h+3
    // (lane = 8 * piece + row).  V, with .trans: at head_dim 64 32 rows x one piece (lane = row); at 128
    // 16 rows x two neighbouring pieces (lane = 16 * piece + row).
    constexpr int KH = HD / 32;   // K instructions per 8-row tile
    uint32_t k_off[KH];
#pragma unroll
    for (int h = 0; h < KH; ++h) {
        const int p = h * 4 + (lane >> 3);
        k_off[h] = (p >> 3) * BOX_BYTES + (lane & 7) * 128 + (((p & 7) ^ (lane & 7)) << 4);
    }
    const int v_r = HD == 64 ? lane : (lane & 15);        // V row this lane addresses
    const int v_p = HD == 64 ? 0 : (lane >> 4);           // ... and which piece of the instruction's pair
    bool alive = true;
    for (int item = first; alive && item < n_items; item += stride) {
        const Work w = decode_work<ROWS>(item, a);
        // count this item in on its sequence's counter once its read of the length has returned (the
        // increment is computed from the value read); the result is looked at when the item is done
        int seq_arrival = -1;
        if (lane == 0) {
            int one;
            asm volatile("and.b32 %0, %1, 0;\n\tadd.s32 %0, %0, 1;" : "=r"(one) : "r"(w.n0));
            seq_arrival = atomicAdd(a.counters + (size_t)a.B * a.H + w.b, one);
        }
        // Q as A fragments (rows g < m; the rest of the 16-row tile is zero)
        uint32_t qa[HD / 16][2];
        {
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(reinterpret_cast<const bf16*>(a.q) + ((size_t)w.bh * a.m + g) * HD);
#pragma unroll
            for (int kk = 0; kk < HD / 16; ++kk) {
                qa[kk][0] = g < a.m ? qrow[kk * 8 + t] : 0u;
                qa[kk][1] = g < a.m ? qrow[kk * 8 + 4 + t] : 0u;
            }
        }
        // query g sees rows below `limit`
        const int limit = w.append ? (g < a.m ? w.n0 + g + 1 : w.n) : w.n0;
        const int full_below = w.append ? w.n0 + 1 : w.n0;   // chunks ending at or below this row need no mask
        float m_run = kNegInf, l_run = 0.f;
        float o[HD / 8][4];
#pragma unroll
        for (int nd = 0; nd < HD / 8; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;

        for (int c = 0; c < w.nchunks; ++c) {
            const uint32_t sidx = consumed % kStages;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8 * sidx, (consumed / kStages) & 1))) {  // warp-uniform outcome
                alive = false;
                break;
            }
            const int row_base = c * ROWS;
            const uint32_t ks = ring0 + sidx * STAGE_BYTES, vs = ks + CHUNK_BYTES;
            const int nvalid = min(ROWS, w.n - row_base);
            if (nvalid < ROWS) {
                // rows past the length may hold anything, and 0 x NaN is NaN: clear their V rows
                for (int i = lane; i < NBOX * (ROWS - nvalid) * 8; i += 32) {
                    const int bx = i / ((ROWS - nvalid) * 8), j = i - bx * ((ROWS - nvalid) * 8);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs + bx * BOX_BYTES + (nvalid + (j >> 3)) * 128 + ((j & 7) << 4)), "r"(0u) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the stage is later rewritten by the copy engine
                __syncwarp();
            }
            constexpr int NV = CHUNK_BYTES / 512;   // V instructions per chunk (512 bytes each)
            uint32_t kb[ROWS / 8][KH][4], vb[NV][4];
#pragma unroll
            for (int nt = 0; nt < ROWS / 8; ++nt)
#pragma unroll
                for (int h = 0; h < KH; ++h) ldmatrix_x4(ks + nt * 1024 + k_off[h], kb[nt][h]);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                // head_dim 64: piece i of rows 0..31 (k-steps 0 and 1 of column tile i);
                // head_dim 128: pieces 2i and 2i+1 of rows 0..15 (column tiles 2i and 2i+1)
                const int p = HD == 64 ? i : 2 * i + v_p;
                ldmatrix_x4_trans(vs + (p >> 3) * BOX_BYTES + v_r * 128 + (((p & 7) ^ (v_r & 7)) << 4), vb[i]);
            }
            // the fragments are in registers: hand the stage back and request the next chunk
            ++consumed;
#pragma unroll
            for (int nt = 0; nt < ROWS / 8; ++nt) asm volatile("" ::"r"(kb[nt][0][0]), "r"(kb[nt][KH - 1][3]) : "memory");
#pragma unroll
            for (int i = 0; i < NV; ++i) asm volatile("" ::"r"(vb[i][0]), "r"(vb[i][3]) : "memory");
            __syncwarp();
            issue_one();

            // S = Q K^T: ROWS / 8 column tiles of 8 rows, HD / 16 k-steps of 16 dims
            float s[ROWS / 8][4];
#pragma unroll
            for (int nt = 0; nt < ROWS / 8; ++nt) {
                s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
                for (int h = 0; h < KH; ++h) {
                    mma_rows0to7(s[nt], qa[2 * h][0], qa[2 * h][1], kb[nt][h][0], kb[nt][h][1]);
                    mma_rows0to7(s[nt], qa[2 * h + 1][0], qa[2 * h + 1][1], kb[nt][h][2], kb[nt][h][3]);
                }
            }
            if (row_base + ROWS > full_below) {   // warp-uniform: the chunk reaches rows some query must not see
#pragma unroll
                for (int nt = 0; nt < ROWS / 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e)
                        if (row_base + nt * 8 + 2 * t + e >= limit) s[nt][e] = kNegInf;
            }
            float mx = kNegInf;
#pragma unroll
            for (int nt = 0; nt < ROWS / 8; ++nt) mx = fmaxf(mx, fmaxf(s[nt][0], s[nt][1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run, mx * a.scale_log2);
            const float m_use = m_new == kNegInf ? 0.f : m_new;   // nothing visible yet: every weight is 0
            const float cf = ex2(m_run - m_use);
            float psum = 0.f;
#pragma unroll
            for (int nt = 0; nt < ROWS / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p = ex2(fmaf(s[nt][e], a.scale_log2, -m_use));
                    psum += p;
                    s[nt][e] = p;
                }
            l_run = l_run * cf + psum;   // this lane's columns only; the four lanes of a row add up at the end
            m_run = m_new;
#pragma unroll
            for (int nd = 0; nd < HD / 8; ++nd) {
                o[nd][0] *= cf;
                o[nd][1] *= cf;
            }
            // O += P V: the score tiles 2k, 2k+1 are the A fragment of k-step k
            uint32_t pa[ROWS / 16][2];
#pragma unroll
            for (int k2 = 0; k2 < ROWS / 16; ++k2) {
                pa[k2][0] = pack_bf16(s[2 * k2][0], s[2 * k2][1]);
                pa[k2][1] = pack_bf16(s[2 * k2 + 1][0], s[2 * k2 + 1][1]);
            }
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                if constexpr (HD == 64) {
                    mma_rows0to7(o[i], pa[0][0], pa[0][1], vb[i][0], vb[i][1]);
                    mma_rows0to7(o[i], pa[1][0], pa[1][1], vb[i][2], vb[i][3]);
                } else {
                    mma_rows0to7(o[2 * i], pa[0][0], pa[0][1], vb[i][0], vb[i][1]);
                    mma_rows0to7(o[2 * i + 1], pa[0][0], pa[0][1], vb[i][2], vb[i][3]);
                }
            }
        }
        if (!alive) break;
        float l = l_run;
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if (g < a.m) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
            uint32_t* orow = reinterpret_cast<uint32_t*>(reinterpret_cast<bf16*>(a.out) + ((size_t)w.bh * a.m + g) * HD);
#pragma unroll
            for (int nd = 0; nd < HD / 8; ++nd) orow[nd * 4 + t] = pack_bf16(o[nd][0] * inv, o[nd][1] * inv);
        }
        if (lane == 0) {
            if ((w.bh % a.H) == 0) {
                if (w.n == 0) raise_status(a.dev_status, BT_DEV_EMPTY);
                if (w.overflow) raise_status(a.dev_status, BT_DEV_OVERFLOW);
            }
            if (seq_arrival == a.H - 1) {   // the last of the sequence's items to have read the old length
                if (w.append) a.len[w.b] = w.n;
                a.counters[(size_t)a.B * a.H + w.b] = 0;
            }
        }
    }
    if (!alive) {
        // a copy never completed: report it, give the copies still in flight one more bounded wait so
        // that none lands in shared memory after the CTA is gone, and leave
        if (lane == 0) raise_status(a.dev_status, BT_DEV_TIMEOUT);
        for (; consumed < issued; ++consumed)
            if (!mbar_wait_bounded(bar0 + 8 * (consumed % kStages), (consumed / kStages) & 1)) break;
    }
}

}  // namespace mq

bool multi_decode_supported(const MultiDecodeArgs& a)
{
    auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return (a.hd == 64 || a.hd == 128) && a.m >= 1 && a.m <= 8 && a.n_max >= 32 && al(a.q) && al(a.k) && al(a.v) && al(a.k_new) && al(a.v_new) && al(a.out) &&
           tensor_map_encode_fn() != nullptr;
}

template <int HD>
static cudaError_t launch_multi_t(const MultiDecodeArgs& a, cudaStream_t stream)
{
    using namespace mq;
    static PerDeviceOnce limit_raised;
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    e = raise_smem_limit_once(limit_raised, dev, block_decode_mq_kernel<HD>, kSmemBytes);
    if (e != cudaSuccess) return e;
    const long long items = (long long)a.B * a.H;
    if (items > 0x7fffffffLL - 4096) return cudaErrorInvalidConfiguration;
    CUtensorMap mk, mv;
    if (!make_slab_map(&mk, a.k, HD, a.n_max, a.n_max, items, Geo<HD>::ROWS) ||
        !make_slab_map(&mv, a.v, HD, a.n_max, a.n_max, items, Geo<HD>::ROWS))
        return cudaErrorInvalidValue;
    const long long grid = items < sms ? items : sms;
    return launch_pdl(block_decode_mq_kernel<HD>, dim3((unsigned)grid), dim3(kThreads), (size_t)kSmemBytes, stream, mk, mv, a);
}

cudaError_t launch_block_decode_multi(const MultiDecodeArgs& a, cudaStream_t stream)
{
    return a.hd == 64 ? launch_multi_t<64>(a, stream) : launch_multi_t<128>(a, stream);
}

}  // namespace bt
