// Block-decoder decode attention (paper section 2.3; appendix E.2), streaming form: the kernel
// is bound by how many bytes of K and V it keeps in flight, so the bytes are moved by the bulk-copy
// engine into shared-memory rings and the warps only compute.
//
// One persistent CTA per SM, six to nine warps (picked per launch).  Every warp works alone: it owns
// a ring of two or three 8 KB stages (depth picked per launch; one stage = a chunk of K rows and the
// same rows of V), takes whole work items ((sequence, head) or (sequence, head, split)), and lane 0
// re-requests a stage with cp.async.bulk as soon as its rows are in registers - across item
// boundaries, so the stream never drains.  No CTA-wide synchronisation exists; a stage is handed back by __syncwarp.  Per chunk a
// lane group of hd/8 lanes owns a row: 128-bit shared-memory reads, fp32 dot product reduced by
// shuffles, online softmax in the log2 domain per lane; row groups merge by shuffles at the end of
// the item.  Every wait on a copy is bounded and raises BT_DEV_TIMEOUT when it runs out.
//
// Two things ride along so that a decode step is one launch per layer.  (1) Split row ranges: every
// item writes its normalised partial and log2-sum-exp, then counts itself in; the item that arrives
// last for a (sequence, head) folds all partials by the log-sum-exp rule and writes the output, so
// no merge launch follows.  (2) Fused append: when a new row is passed in, the item that owns the
// last row takes it from the caller's buffer (and stores it into the cache) instead of streaming
// it; the sequence's length is raised by the item that is last to finish with that sequence, once
// every item has read the old one.  Both counters return to zero before the kernel ends.
#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"

namespace bt {
namespace ring {

#ifndef BT_DEC_WARPS
#define BT_DEC_WARPS 8
#endif
#ifndef BT_DEC_MAX_WARPS
#define BT_DEC_MAX_WARPS 12
#endif
#ifndef BT_DEC_STAGES
#define BT_DEC_STAGES 3
#endif
#ifndef BT_DEC_UNROLL
#define BT_DEC_UNROLL 8
#endif
// Warps per CTA are chosen per launch (kMinWarps..kMaxWarps, kWarps unless another count leaves fewer
// warps idle in the last round of items): every warp has its own ring, so the kernel only needs the count.
constexpr int kWarps = BT_DEC_WARPS;
constexpr int kMinWarps = 6, kMaxWarps = BT_DEC_MAX_WARPS;   // the register budget allows twelve (two-stage rings only)
constexpr int kMaxWarpsLong = 9;      // most warps considered when the rows may be many
constexpr int kShortCacheRows = 320;  // capacity up to which an item is short enough for twelve warps to pay
constexpr int kMaxThreads = kMaxWarps * 32;
// Ring depth, chosen per launch: two stages when at least three warps in four have an item (with the
// memory system saturated by many rings, less in flight per warp runs faster: 82.4 vs 84.2 us at 4096
// items of 512 rows, 158 vs 164 us at 1024 items of 4096 rows), kDeepStages when only some of the warps
// have an item and each must cover more of the latency on its own (27.5 vs 28.7 us at 512 items).
constexpr int kDeepStages = BT_DEC_STAGES;
constexpr int kUnroll = BT_DEC_UNROLL;     // rows per lane group per chunk
constexpr int kPrefetchChunks = 16;         // chunks of a warp's first item warmed in L2 ahead of the dependent-launch wait
constexpr uint32_t kPollLimit = 1u << 24;  // polls of one wait before giving up (each poll suspends briefly)

template <int HD>
struct Geo {
    static constexpr int LPR = RowGeo<HD>::LPR, RPW = RowGeo<HD>::RPW;
    static constexpr int ROWS = kUnroll * RPW;          // rows per chunk: 32 at hd 64, 16 at hd 128
    static constexpr int ROW_BYTES = HD * 2;
    static constexpr int CHUNK_BYTES = ROWS * ROW_BYTES;  // 4096
    static constexpr int STAGE_BYTES = 2 * CHUNK_BYTES;   // K chunk, then V chunk
};
template <int HD>
constexpr int smem_bytes(int warps, int stages) { return warps * stages * Geo<HD>::STAGE_BYTES + warps * stages * 8; }

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) { return mbar_wait_polls(bar, parity, kPollLimit); }
// bytes global -> shared, completion counted on the mbarrier; the rows are read once, so they are
// marked evict-first in L2
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

// Row range of one work item.  n counts the appended row when there is one; rows [r0, c1) come from
// the cache, and row n-1 from the caller's buffer when new_row is set.
struct Work {
    int bh, sp, b, n, r0, c1;
    bool new_row, overflow;
};
// Position of a warp in the line of items: item = bh * splits + sp, bh = b * H + h.  A warp walks the line with a
// fixed stride, so the parts are carried forward by additions (the divisions happen once, in Step): with caches of
// a few dozen rows an item is a thousand instructions, and integer divisions were a sixth of them.
struct Cursor {
    int item, bh, sp, b, h;
};
struct Step {   // stride split into its parts
    int items, bh, sp, b, h;
};
__device__ __forceinline__ Cursor cursor_at(int item, const DecodeArgs& a)
{
    Cursor c;
    c.item = item;
    c.bh = item / a.splits;
    c.sp = item - c.bh * a.splits;
    c.b = c.bh / a.H;
    c.h = c.bh - c.b * a.H;
    return c;
}
__device__ __forceinline__ Step step_of(int stride, const DecodeArgs& a)
{
    Step s;
    s.items = stride;
    s.bh = stride / a.splits;
    s.sp = stride - s.bh * a.splits;
    s.b = s.bh / a.H;
    s.h = s.bh - s.b * a.H;
    return s;
}
__device__ __forceinline__ void advance(Cursor& c, const Step& s, const DecodeArgs& a)
{
    c.item += s.items;
    c.sp += s.sp;
    const int carry_sp = c.sp >= a.splits ? 1 : 0;
    c.sp -= carry_sp ? a.splits : 0;
    c.bh += s.bh + carry_sp;
    c.h += s.h + carry_sp;              // < 2 H
    const int carry_h = c.h >= a.H ? 1 : 0;
    c.h -= carry_h ? a.H : 0;
    c.b += s.b + carry_h;
}
__device__ __forceinline__ Work decode_work(const Cursor& c, const DecodeArgs& a)
{
    Work w;
    w.bh = c.bh;
    w.sp = c.sp;
    w.b = c.b;
    int n = a.len[w.b];
    n = n < 0 ? 0 : (n > a.n_max ? a.n_max : n);
    const bool append = a.k_new != nullptr && n < a.n_max;  // a full cache takes no row: flagged, attended as it is
    w.overflow = a.k_new != nullptr && !append;
    n += append ? 1 : 0;
    w.n = n;
    // rows per split, rounded up to whole 32-row groups so that every split starts on a chunk boundary
    // (trailing splits may then be empty)
    const int per = a.splits == 1 ? n : (((n + a.splits - 1) / a.splits + 31) & ~31);
    w.r0 = min(n, w.sp * per);
    const int r1 = min(n, w.r0 + per);
    w.new_row = append && r1 == n && w.r0 < n;   // exactly one split ends at row n-1
    w.c1 = w.new_row ? r1 - 1 : r1;
    return w;
}

// grid: one CTA per SM (fewer when there are fewer items than warps).  splits == 1 writes bf16
// output directly; otherwise each item writes its normalised partial (hd floats, then its
// log2-sum-exp; hd+4 floats apart so that every partial is 16-byte aligned) to the workspace and the
// last one to arrive combines them.
template <int HD, int kStages>
__global__ void __launch_bounds__(kMaxThreads, 1) block_decode_ring_kernel(DecodeArgs a)
{
    using G = Geo<HD>;
    constexpr int LPR = G::LPR, RPW = G::RPW, ROWS = G::ROWS;
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rg = lane / LPR;
    const uint32_t ring0 = smem_u32(smem) + warp * (kStages * G::STAGE_BYTES);
    const int n_warps = blockDim.x >> 5;
    const uint32_t bar0 = smem_u32(smem) + n_warps * kStages * G::STAGE_BYTES + warp * (kStages * 8);

    if (lane == 0) {
        for (int s = 0; s < kStages; ++s)
            mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    pdl_launch_dependents();

    const int n_items = a.B * a.H * a.splits;
    const int stride = n_warps * gridDim.x;
    const int first = warp * gridDim.x + blockIdx.x;   // neighbouring items go to different SMs
    bf16* Kall = reinterpret_cast<bf16*>(a.k);
    bf16* Vall = reinterpret_cast<bf16*>(a.v);
    // While the kernel before this one drains, warm L2 with this warp's first item (up to kPrefetchChunks
    // chunks of it), its length and its query: CTAs that are placed early sit idle until the last CTA
    // of the previous kernel is gone, and HBM is not busy during that tail.  A prefetch returns nothing
    // to the thread, so it is safe ahead of the wait.  How many rows to touch comes from a look at the
    // length that may be out of date (read past L1, so that no stale copy stays behind for the read
    // after the wait): it is only a hint for the prefetch and never decides what is computed.
    if (first < n_items && a.splits == 1) {
        int n_hint = __ldcg(a.len + first / a.H);
        n_hint = n_hint < 0 ? 0 : (n_hint >= a.n_max ? a.n_max : n_hint + 1);
        const size_t off = (size_t)first * a.n_max * HD;
        const int lines = (min(kPrefetchChunks * G::CHUNK_BYTES, n_hint * G::ROW_BYTES) + 127) / 128;  // 128-byte lines to touch
        for (int i = lane; i < lines; i += 32) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Kall + off) + (size_t)i * 128));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Vall + off) + (size_t)i * 128));
        }
        if (lane == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const bf16*>(a.q) + (size_t)first * HD));
    }
    pdl_wait();  // nothing above wrote global memory, or used a value read from it for more than a prefetch hint

    // ---- producer cursor (kept by every lane, acted on by lane 0): next chunk to request
    const Step step = step_of(stride, a);
    Cursor pc = cursor_at(first < n_items ? first : 0, a);
    pc.item = first;
    int p_c = 0, p_nchunks = 0;
    Work pw = {};
    auto p_seek = [&]() {  // move to the next item that has rows
        while (pc.item < n_items) {
            pw = decode_work(pc, a);
            p_nchunks = (pw.c1 - pw.r0 + ROWS - 1) / ROWS;
            if (p_nchunks > 0) {
                p_c = 0;
                return;
            }
            advance(pc, step, a);
        }
    };
    uint32_t issued = 0, consumed = 0;
    auto issue_one = [&]() {
        if (pc.item >= n_items) return;
        const int row = pw.r0 + p_c * ROWS;
        const uint32_t bytes = (uint32_t)min(ROWS, pw.c1 - row) * G::ROW_BYTES;
        const uint32_t st = issued % kStages;
        if (lane == 0) {
            const uint32_t bar = bar0 + 8 * st, dst = ring0 + st * G::STAGE_BYTES;
            const size_t off = ((size_t)pw.bh * a.n_max + row) * HD;
            mbar_expect_tx(bar, 2 * bytes);
            bulk_load(dst, Kall + off, bytes, bar, policy);
            bulk_load(dst + G::CHUNK_BYTES, Vall + off, bytes, bar, policy);
        }
        ++issued;
        if (++p_c == p_nchunks) {
            advance(pc, step, a);
            p_seek();
        }
    };
    p_seek();
    for (int s = 0; s < kStages; ++s) issue_one();

    // ---- consumer: whole items, chunk by chunk
    bool alive = true;
    const bf16* Qall = reinterpret_cast<const bf16*>(a.q);
    uint4 q_next = make_uint4(0, 0, 0, 0);  // the query of the next item is fetched an item ahead
    // ... and so is the row to append (whichever item of the (sequence, head) turns out to own it: the loads are
    // speculative and cost 2 x 16 bytes per lane group).  With caches of a few dozen rows an item is over sooner
    // than a round trip to DRAM, so nothing an item needs may be requested inside it.
    uint4 kn_next = make_uint4(0, 0, 0, 0), vn_next = kn_next;
    Cursor cc = cursor_at(first < n_items ? first : 0, a);   // this item
    cc.item = first;
    Cursor cn = cc;                                          // the item after it
    advance(cn, step, a);
    if (first < n_items) {
        q_next = ld_plain(Qall + (size_t)cc.bh * HD + sub * 8);
        if (a.k_new != nullptr) {
            kn_next = ld_plain(reinterpret_cast<const bf16*>(a.k_new) + (size_t)cc.bh * HD + sub * 8);
            vn_next = ld_plain(reinterpret_cast<const bf16*>(a.v_new) + (size_t)cc.bh * HD + sub * 8);
        }
    }
    // The length update of an item is settled one item later, for the same reason: the count it depends on comes
    // back from L2.  (lane 0 only)
    int pend_arrival = -1, pend_b = 0, pend_n = 0;
    bool pend_overflow = false;
    auto settle = [&]() {
        if (pend_arrival == a.H * a.splits - 1) {
            // that item was the last of its sequence to read the old length: raise it
            if (!pend_overflow) a.len[pend_b] = pend_n;
            a.counters[(size_t)a.B * a.H + pend_b] = 0;
        }
    };
    for (; alive && cc.item < n_items; cc = cn, advance(cn, step, a)) {
        const Work w = decode_work(cc, a);
        // Fused append: the sequence's length goes up once all of its H * splits items have read the old
        // one.  An item counts itself in as soon as its own read has returned (the increment is computed
        // from the value read, so the count cannot be issued before that) and looks at the result only
        // when it is done, a whole item later: nothing ever waits for the round trip.  Whoever counted in
        // last raises the length.  (This warp's look-ahead read of the same length came even earlier.)
        int seq_arrival = -1;
        if (a.k_new != nullptr && lane == 0) {
            int one;
            asm volatile("and.b32 %0, %1, 0;\n\tadd.s32 %0, %0, 1;" : "=r"(one) : "r"(w.n));
            seq_arrival = atomicAdd(a.counters + (size_t)a.B * a.H + w.b, one);
        }
        float qf[8];
        {
            const uint4 qr = q_next;
            if (cn.item < n_items) q_next = ld_plain(Qall + (size_t)cn.bh * HD + sub * 8);
            unpack8(qr, qf);
#pragma unroll
            for (int i = 0; i < 8; ++i) qf[i] *= a.scale_log2;
        }
        // the row to append (used only if this item owns it), fetched an item ago; the next item's is requested now
        const uint4 kn = kn_next, vn = vn_next;
        if (a.k_new != nullptr && cn.item < n_items) {
            const size_t nb = (size_t)cn.bh * HD + sub * 8;
            kn_next = ld_plain(reinterpret_cast<const bf16*>(a.k_new) + nb);
            vn_next = ld_plain(reinterpret_cast<const bf16*>(a.v_new) + nb);
        }
        SoftmaxState st;
        st.init();
        const int nchunks = (w.c1 - w.r0 + ROWS - 1) / ROWS;
        for (int c = 0; c < nchunks; ++c) {
            const uint32_t sidx = consumed % kStages;
            // the outcome is made warp-uniform: the shuffles and __syncwarp below need all 32 lanes
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8 * sidx, (consumed / kStages) & 1))) {
                alive = false;
                break;
            }
            const int nvalid = min(ROWS, w.c1 - (w.r0 + c * ROWS));
            const uint32_t ks = ring0 + sidx * G::STAGE_BYTES + rg * G::ROW_BYTES + sub * 16;
            const uint32_t vs = ks + G::CHUNK_BYTES;
            uint4 kr[kUnroll], vr[kUnroll];
            float s[kUnroll];
            float mt = kNegInf;
            auto refill = [&]() {
                ++consumed;
                // the loaded values must be in registers, not merely requested, before the stage is overwritten
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) asm volatile("" ::"r"(kr[u].x), "r"(vr[u].x) : "memory");
                __syncwarp();
                issue_one();
            };
            if (nvalid == ROWS) {
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) kr[u] = lds128(ks + u * RPW * G::ROW_BYTES);
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) vr[u] = lds128(vs + u * RPW * G::ROW_BYTES);
                refill();   // the rows are in registers: request the next chunk before the arithmetic
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    s[u] = row_sum<LPR>(dot8(qf, kr[u]));
                    mt = fmaxf(mt, s[u]);
                }
            } else {  // ragged tail: rows past the range were not copied and count as absent
                const uint4 zero = make_uint4(0, 0, 0, 0);
                const int ngroups = (nvalid + RPW - 1) / RPW;   // groups of RPW rows that hold any row at all (warp-uniform)
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const bool valid = u * RPW + rg < nvalid;
                    kr[u] = valid ? lds128(ks + u * RPW * G::ROW_BYTES) : zero;
                    vr[u] = valid ? lds128(vs + u * RPW * G::ROW_BYTES) : zero;
                }
                refill();
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    s[u] = kNegInf;
                    if (u < ngroups) {
                        const float d = row_sum<LPR>(dot8(qf, kr[u]));
                        s[u] = (u * RPW + rg < nvalid) ? d : kNegInf;
                        mt = fmaxf(mt, s[u]);
                    }
                }
                if (mt != kNegInf) {  // uniform within the LPR lanes of a row group
                    const float mn = fmaxf(st.m, mt);
                    const float cf = ex2(st.m - mn);
                    st.l *= cf;
#pragma unroll
                    for (int i = 0; i < 8; ++i) st.acc[i] *= cf;
#pragma unroll
                    for (int u = 0; u < kUnroll; ++u) {
                        if (u < ngroups) {
                            const float p = ex2(s[u] - mn);   // 0 for the absent rows of the last group
                            st.l += p;
                            fma8(st.acc, p, vr[u]);
                        }
                    }
                    st.m = mn;
                }
                continue;
            }
            if (mt != kNegInf) {  // uniform within the LPR lanes of a row group
                const float mn = fmaxf(st.m, mt);
                const float cf = ex2(st.m - mn);
                st.l *= cf;
#pragma unroll
                for (int i = 0; i < 8; ++i) st.acc[i] *= cf;
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const float p = ex2(s[u] - mn);
                    st.l += p;
                    fma8(st.acc, p, vr[u]);
                }
                st.m = mn;
            }
        }
        if (!alive) break;
        if (w.new_row) {  // warp-uniform.  Row n-1 = the new row: scored from registers, stored into the cache
            const float sn = row_sum<LPR>(dot8(qf, kn));
            if (rg == 0) {
                const float mn = fmaxf(st.m, sn);
                const float cf = ex2(st.m - mn), pn = ex2(sn - mn);
                st.l = st.l * cf + pn;
#pragma unroll
                for (int i = 0; i < 8; ++i) st.acc[i] *= cf;
                fma8(st.acc, pn, vn);
                st.m = mn;
                const size_t off = ((size_t)w.bh * a.n_max + (w.n - 1)) * HD + sub * 8;
                *reinterpret_cast<uint4*>(Kall + off) = kn;
                *reinterpret_cast<uint4*>(Vall + off) = vn;
            }
        }
        // merge the RPW row groups of the warp
        auto merge_row_groups = [&]() {
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1) {
                const float m2 = __shfl_xor_sync(0xffffffffu, st.m, off);
                const float l2 = __shfl_xor_sync(0xffffffffu, st.l, off);
                float a2[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a2[i] = __shfl_xor_sync(0xffffffffu, st.acc[i], off);
                st.merge(m2, l2, a2);
            }
        };
        auto write_out = [&]() {  // lanes of row group 0: normalised bf16 output row
            float o[8];
            const float inv = st.l > 0.f ? 1.f / st.l : 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = st.acc[i] * inv;
            *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.out) + (size_t)w.bh * HD + sub * 8) = pack8(o);
        };
        merge_row_groups();
        if (a.splits == 1) {
            if (rg == 0) write_out();
        } else {
            if (rg == 0) {
                float o[8];
                const float inv = st.l > 0.f ? 1.f / st.l : 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) o[i] = st.acc[i] * inv;
                float* ws = a.ws + ((size_t)w.bh * a.splits + w.sp) * (HD + 4);
                *reinterpret_cast<float4*>(ws + sub * 8) = make_float4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<float4*>(ws + sub * 8 + 4) = make_float4(o[4], o[5], o[6], o[7]);
                if (sub == 0) ws[HD] = st.l > 0.f ? st.m + log2f(st.l) : kNegInf;
                __threadfence();  // the partial is visible before this item counts itself in
            }
            __syncwarp();
            int last = 0;
            if (lane == 0) last = atomicAdd(a.counters + w.bh, 1) == a.splits - 1;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {  // every split of (b,h) has written: fold the partials (normalised, weight 2^lse each)
                __threadfence();
                st.init();
                for (int s2 = rg; s2 < a.splits; s2 += RPW) {
                    const float* ws = a.ws + ((size_t)w.bh * a.splits + s2) * (HD + 4);
                    const float lse = __ldcg(ws + HD);
                    const float4 x = __ldcg(reinterpret_cast<const float4*>(ws + sub * 8));
                    const float4 y = __ldcg(reinterpret_cast<const float4*>(ws + sub * 8 + 4));
                    const float a2[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
                    st.merge(lse, 1.f, a2);
                }
                merge_row_groups();
                if (rg == 0) write_out();
                if (lane == 0) a.counters[w.bh] = 0;
            }
        }
        if (w.sp == 0 && cc.h == 0 && lane == 0) {
            if (w.n == 0) raise_status(a.dev_status, BT_DEV_EMPTY);
            if (w.overflow) raise_status(a.dev_status, BT_DEV_OVERFLOW);
        }
        settle();   // the item before this one: its count has long come back
        pend_arrival = seq_arrival;
        pend_b = w.b;
        pend_n = w.n;
        pend_overflow = w.overflow;
    }
    settle();
    if (!alive) {
        // a copy never completed: report it, give the copies still in flight one more bounded wait so
        // that none lands in shared memory after the CTA is gone, and leave
        if (lane == 0) raise_status(a.dev_status, BT_DEV_TIMEOUT);
        for (; consumed < issued; ++consumed)
            if (!mbar_wait_bounded(bar0 + 8 * (consumed % kStages), (consumed / kStages) & 1)) break;
    }
}

template <int HD, int STAGES>
static cudaError_t launch_st(const DecodeArgs& a, long long grid, int warps, int dev, cudaStream_t stream)
{
    static PerDeviceOnce limit_raised;
    cudaError_t e = raise_smem_limit_once(limit_raised, dev, block_decode_ring_kernel<HD, STAGES>, smem_bytes<HD>(STAGES == 2 ? kMaxWarps : kMaxWarpsLong, STAGES));
    if (e != cudaSuccess) return e;
    return launch_pdl(block_decode_ring_kernel<HD, STAGES>, dim3((unsigned)grid), dim3(warps * 32),
                      (size_t)smem_bytes<HD>(warps, STAGES), stream, a);
}

template <int HD>
static cudaError_t launch_t(const DecodeArgs& a, cudaStream_t stream)
{
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    const long long items = (long long)a.B * a.H * a.splits;
    if (items > 0x7fffffffLL - 4096) return cudaErrorInvalidConfiguration;
    // one CTA per SM; with few items, one item per CTA first so that they spread over the SMs
    long long grid = items < sms ? items : sms;
    // Items are dealt whole, so the launch takes ceil(items / warps) rounds and the warps of the last round
    // that have no item idle while a warp cannot stream faster than its ring allows: pick the warp count
    // with the fullest last round (4096 items on 148 SMs: 7 warps run 3.95 -> 4 rounds, 8 warps 3.46 -> 4).
    int warps = kWarps;
    double best = 0.0;
    for (int w = kMaxWarpsLong; w >= kMinWarps; --w) {
        const long long slots = grid * w, rounds = (items + slots - 1) / slots;
        const double fill = (double)items / (double)(rounds * slots) + (w == kWarps ? 1e-9 : 0.0);  // ties go to kWarps
        if (fill > best) {
            best = fill;
            warps = w;
        }
    }
    // Short caches (the capacity bounds the rows): an item is then about a thousand instructions whatever its rows,
    // and what limits the launch is how many warps an SM has to interleave - twelve when all of them get items
    // (17.7 vs 21.6 us at 8192 items of 17 rows; at 272 rows the same, at 512 rows eight warps win).
    if (a.n_max <= kShortCacheRows && items >= grid * kMaxWarps) warps = kMaxWarps;
    const bool shallow = items * 4 >= grid * warps * 3 || warps > kMaxWarpsLong;   // (nearly) every warp has an item: the shallow ring
    return shallow ? launch_st<HD, 2>(a, grid, warps, dev, stream) : launch_st<HD, kDeepStages>(a, grid, warps, dev, stream);
}

}  // namespace ring

cudaError_t launch_block_decode(const DecodeArgs& a, cudaStream_t stream)
{
    return a.hd == 64 ? ring::launch_t<64>(a, stream) : ring::launch_t<128>(a, stream);
}

}  // namespace bt
