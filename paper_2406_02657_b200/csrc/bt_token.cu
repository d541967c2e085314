// Fused token-decoder step (paper section 2.4; appendix E.2): block-boundary reset, append of
// the new K,V rows to the local cache and attention confined to the current block, in one
// launch over thousands of sequences.  A group of LPR = hd/8 lanes owns one (sequence, head):
// each lane holds 16 bytes of every row, so the whole step is a handful of independent 128-bit
// loads, a few shuffles and one 128-bit store per tensor.  A CTA always covers whole sequences
// so that every head reads the old length before one thread writes the new one.
#include "bt_common.cuh"
#include "bt_device.h"
#include "bt_kernels.h"

namespace bt {

// online-softmax update of one lane group with one row
__device__ __forceinline__ void add_row(SoftmaxState& st, float s, const uint4& vrow)
{
    float mn = fmaxf(st.m, s);
    float c = ex2(st.m - mn), p = ex2(s - mn);
    st.l = st.l * c + p;
#pragma unroll
    for (int i = 0; i < 8; ++i) st.acc[i] *= c;
    fma8(st.acc, p, vrow);
    st.m = mn;
}

#ifndef BT_TOK_X2
#define BT_TOK_X2 1
#endif
#ifndef BT_TOK_MINBLOCKS
#define BT_TOK_MINBLOCKS 3
#endif
#ifndef BT_TOK_THREADS
#define BT_TOK_THREADS 256
#endif

template <int HD>
__global__ void __launch_bounds__(256, BT_TOK_MINBLOCKS) token_decode_kernel(TokenArgs a, int seqs_per_cta, int threads_per_seq)
{
    constexpr int LPR = RowGeo<HD>::LPR;
    const int tid = threadIdx.x;
    const int sic = tid / threads_per_seq;            // sequence within the CTA
    const int within = tid - sic * threads_per_seq;
    const int h = within / LPR, sub = within % LPR;
    const int b = blockIdx.x * seqs_per_cta + sic;
    const bool active = sic < seqs_per_cta && b < a.B;

    pdl_launch_dependents();  // launched with launch_pdl
    pdl_wait();               // nothing above touched global memory
    const bool appended = a.k_new != nullptr;
    const bool fast = a.n_q == 1 && appended;
    const size_t slab = active ? (size_t)b * a.H + h : 0;
    bf16* cache = reinterpret_cast<bf16*>(a.kv) + slab * a.cap * 2 * HD + sub * 8;  // row r: K at +r*2*HD, V at +(r*2+1)*HD
    const bf16* qp = reinterpret_cast<const bf16*>(a.q) + slab * a.n_q * HD + sub * 8;
    const bf16* kp = reinterpret_cast<const bf16*>(a.k_new) + slab * a.n_q * HD + sub * 8;
    const bf16* vp = reinterpret_cast<const bf16*>(a.v_new) + slab * a.n_q * HD + sub * 8;
    bf16* op = reinterpret_cast<bf16*>(a.out) + slab * a.n_q * HD + sub * 8;

    // the new row does not depend on the length: get it in flight before the length arrives
    uint4 qr = make_uint4(0, 0, 0, 0), kr = qr, vr = qr;
    if (fast && active) {
        qr = ld_stream(qp);
        kr = ld_stream(kp);
        vr = ld_stream(vp);
    }
    int len_old = 0;
    if (active) {
        const bool rst = a.reset_mask ? (a.reset_mask[b] != 0) : (a.reset_first != 0);
        len_old = rst ? 0 : a.len[b];
    }
    __syncthreads();  // every head has read len[b] before the leader overwrites it

    const bool overflow = appended && (len_old < 0 || len_old + a.n_q > a.cap);
    if (len_old < 0) len_old = 0;
    if (len_old > a.cap) len_old = a.cap;

    if (fast) {
        // token step: the new row stays in registers, the cached rows are read once
        const int n_old = (active && !overflow) ? len_old : 0;
        float qf[8];
        unpack8(qr, qf);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[i] *= a.scale_log2;
        SoftmaxState st;
        st.init();
        for (int j0 = 0; j0 < a.cap; j0 += 4) {  // uniform trip count: shuffles stay convergent
            uint4 kc[4], vc[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool v = j0 + u < n_old;
                kc[u] = v ? ld_stream(cache + (size_t)(j0 + u) * 2 * HD) : make_uint4(0, 0, 0, 0);
                vc[u] = v ? ld_stream(cache + (size_t)(j0 + u) * 2 * HD + HD) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float s = row_sum<LPR>(dot8(qf, kc[u]));
                if (j0 + u < n_old) add_row(st, s, vc[u]);
            }
        }
        float s_new = row_sum<LPR>(dot8(qf, kr));
        if (active && !overflow) {
            *reinterpret_cast<uint4*>(cache + (size_t)len_old * 2 * HD) = kr;
            *reinterpret_cast<uint4*>(cache + (size_t)len_old * 2 * HD + HD) = vr;
            add_row(st, s_new, vr);
        }
        if (active) {
            float o[8];
            float inv = st.l > 0.f ? 1.f / st.l : 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = st.acc[i] * inv;
            *reinterpret_cast<uint4*>(op) = pack8(o);
        }
    } else {
        // general step: n_q rows (the P prefix rows at a block start), or attend-only (n_q queries over rows
        // that a projection has already cached).
        // New rows are written first; each lane later re-reads only bytes it wrote itself.
        if (active && appended && !overflow)
            for (int i = 0; i < a.n_q; ++i) {
                *reinterpret_cast<uint4*>(cache + (size_t)(len_old + i) * 2 * HD) = ld_stream(kp + (size_t)i * HD);
                *reinterpret_cast<uint4*>(cache + (size_t)(len_old + i) * 2 * HD + HD) = ld_stream(vp + (size_t)i * HD);
            }
        for (int i = 0; i < a.n_q; ++i) {
            uint4 qr = active ? ld_stream(qp + (size_t)i * HD) : make_uint4(0, 0, 0, 0);
            float qf[8];
            unpack8(qr, qf);
#pragma unroll
            for (int d = 0; d < 8; ++d) qf[d] *= a.scale_log2;
            // attend only: the queries are those of the last n_q cached rows, the same causal rule counted from the end
            const int n = (!active || overflow) ? 0 : (appended ? len_old + i + 1 : len_old - a.n_q + i + 1);
            SoftmaxState st;
            st.init();
            for (int j = 0; j < a.cap; ++j) {
                const bool v = j < n;
                uint4 kc = v ? ld_plain(cache + (size_t)j * 2 * HD) : make_uint4(0, 0, 0, 0);
                uint4 vc = v ? ld_plain(cache + (size_t)j * 2 * HD + HD) : make_uint4(0, 0, 0, 0);
                float s = row_sum<LPR>(dot8(qf, kc));
                if (v) add_row(st, s, vc);
            }
            if (active) {
                float o[8];
                float inv = st.l > 0.f ? 1.f / st.l : 0.f;
#pragma unroll
                for (int d = 0; d < 8; ++d) o[d] = st.acc[d] * inv;
                *reinterpret_cast<uint4*>(op + (size_t)i * HD) = pack8(o);
            }
        }
    }

    if (active && within == 0) {
        if (overflow) {
            raise_status(a.dev_status, BT_DEV_OVERFLOW);  // sequence skipped, length unchanged
        } else {
            a.len[b] = appended ? len_old + a.n_q : len_old;
            if (!appended && len_old < a.n_q) raise_status(a.dev_status, BT_DEV_EMPTY);  // a query with nothing to see
        }
    }
}

// Block start (section 2.4): every sequence is reset and its P prefix rows arrive together, n_q = P <= kMaxQ.
// There is nothing cached to read: all 3 P rows are requested at once and stay in registers, query i attends
// to the new rows 0..i, the rows go to cache rows 0..P-1 and the length becomes P.  Same thread layout as the
// general kernel (hd/8 lanes per (sequence, head), whole sequences per CTA).
template <int HD, int kMaxQ>
__global__ void __launch_bounds__(256) token_block_start_kernel(TokenArgs a, int seqs_per_cta, int threads_per_seq)
{
    constexpr int LPR = RowGeo<HD>::LPR;
    const int tid = threadIdx.x;
    const int sic = tid / threads_per_seq;
    const int within = tid - sic * threads_per_seq;
    const int h = within / LPR, sub = within % LPR;
    const int b = blockIdx.x * seqs_per_cta + sic;
    const bool active = sic < seqs_per_cta && b < a.B;
    pdl_launch_dependents();
    pdl_wait();
    const size_t slab = active ? (size_t)b * a.H + h : 0;
    bf16* cache = reinterpret_cast<bf16*>(a.kv) + slab * a.cap * 2 * HD + sub * 8;
    const bf16* qp = reinterpret_cast<const bf16*>(a.q) + slab * a.n_q * HD + sub * 8;
    const bf16* kp = reinterpret_cast<const bf16*>(a.k_new) + slab * a.n_q * HD + sub * 8;
    const bf16* vp = reinterpret_cast<const bf16*>(a.v_new) + slab * a.n_q * HD + sub * 8;
    bf16* op = reinterpret_cast<bf16*>(a.out) + slab * a.n_q * HD + sub * 8;
    uint4 qn[kMaxQ], kn[kMaxQ], vn[kMaxQ];
#pragma unroll
    for (int i = 0; i < kMaxQ; ++i) {
        const bool v = active && i < a.n_q;
        qn[i] = v ? ld_stream(qp + (size_t)i * HD) : make_uint4(0, 0, 0, 0);
        kn[i] = v ? ld_stream(kp + (size_t)i * HD) : make_uint4(0, 0, 0, 0);
        vn[i] = v ? ld_stream(vp + (size_t)i * HD) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < kMaxQ; ++i) {
        if (i < a.n_q) {  // uniform
            float qf[8];
            unpack8(qn[i], qf);
#pragma unroll
            for (int d = 0; d < 8; ++d) qf[d] *= a.scale_log2;
            float sc[kMaxQ];
            float mx = kNegInf;
#pragma unroll
            for (int j = 0; j < kMaxQ; ++j) {
                if (j <= i) {
                    sc[j] = row_sum<LPR>(dot8(qf, kn[j]));
                    mx = fmaxf(mx, sc[j]);
                }
            }
            float l = 0.f, acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < kMaxQ; ++j) {
                if (j <= i) {
                    const float pj = ex2(sc[j] - mx);
                    l += pj;
                    fma8(acc, pj, vn[j]);
                }
            }
            if (active) {
                float o[8];
                const float inv = 1.f / l;
#pragma unroll
                for (int d = 0; d < 8; ++d) o[d] = acc[d] * inv;
                *reinterpret_cast<uint4*>(op + (size_t)i * HD) = pack8(o);
                *reinterpret_cast<uint4*>(cache + (size_t)i * 2 * HD) = kn[i];
                *reinterpret_cast<uint4*>(cache + (size_t)i * 2 * HD + HD) = vn[i];
            }
        }
    }
    if (active && within == 0) a.len[b] = a.n_q;  // nobody reads the old length here: the reset drops it
}

// ---------------------------------------------------------------------------------------
// Pipelined token step (n_q = 1 with append: the per-token hot path).  The step is a stream of
// tiny independent problems whose only serial hop is "read the length, then fetch that many
// rows".  A persistent CTA walks groups of whole sequences and keeps kDepth groups in flight:
// each thread copies the 16-byte pieces it will need (q, k_new, v_new and the cached rows below
// the length) with cp.async into shared-memory slots that only it reads back, so no barrier is
// needed for the data, and the lengths are fetched one group further ahead.  The one barrier per
// group orders "every head has read len[b]" before "the leader writes the new len[b]".
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kTokThreads = 256;

template <int HD, int kDepth, int kMaxRows, int kMinBlocks>
__global__ void __launch_bounds__(kTokThreads, kMinBlocks)
token_step_pipelined_kernel(TokenArgs a, int seqs_per_cta, int threads_per_seq)
{
    constexpr int max_rows = kMaxRows;
    constexpr int LPR = RowGeo<HD>::LPR;
    constexpr int kStages = kDepth + 1;
    extern __shared__ uint4 slots_mem[];  // [kStages][3 + 2*max_rows][kTokThreads]
    constexpr int n_slots = 3 + 2 * max_rows;
    const int tid = threadIdx.x;
    const int sic = tid / threads_per_seq;
    const int within = tid - sic * threads_per_seq;
    const int h = within / LPR, sub = within % LPR;
    const bool lane_used = sic < seqs_per_cta;
    const int n_groups = (a.B + seqs_per_cta - 1) / seqs_per_cta;
    const int n_iter = (n_groups - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // same for the whole CTA

    auto seq_of = [&](int i) -> int {
        const int b = ((int)blockIdx.x + i * (int)gridDim.x) * seqs_per_cta + sic;
        return (lane_used && i < n_iter && b < a.B) ? b : -1;
    };
    auto load_len = [&](int b) -> int {
        if (b < 0) return 0;
        const bool rst = a.reset_mask ? (a.reset_mask[b] != 0) : (a.reset_first != 0);
        return rst ? 0 : a.len[b];
    };
    auto slot_addr = [&](int stage, int slot) -> uint32_t {
        return (uint32_t)__cvta_generic_to_shared(slots_mem + ((size_t)stage * n_slots + slot) * kTokThreads + tid);
    };
    // Attend only (k_new == NULL: the step's row was cached by the projection that produced it): nothing is
    // appended, the query sees all len rows, neither the cache nor the length is written.
    const bool appended = a.k_new != nullptr;
    // rows of the cache this thread must fetch for a sequence whose length (before the step) is len
    auto rows_to_read = [&](int len) -> int {
        if (appended) return (len < 0 || len + 1 > a.cap) ? 0 : len;
        return len < 0 ? 0 : (len > max_rows ? max_rows : len);   // the launcher guarantees cap <= max_rows here
    };
    // the new row and the query do not depend on the length ...
    auto issue_new = [&](int i) {
        const int b = seq_of(i);
        if (b >= 0) {
            const int stage = i % kStages;
            const size_t slab = (size_t)b * a.H + h;
            cp_async16(slot_addr(stage, 0), reinterpret_cast<const bf16*>(a.q) + slab * HD + sub * 8);
            if (appended) {
                cp_async16(slot_addr(stage, 1), reinterpret_cast<const bf16*>(a.k_new) + slab * HD + sub * 8);
                cp_async16(slot_addr(stage, 2), reinterpret_cast<const bf16*>(a.v_new) + slab * HD + sub * 8);
            }
        }
    };
    // ... the cached rows to fetch do
    auto issue_rows = [&](int i, int len) {
        const int b = seq_of(i);
        if (b >= 0) {
            const int stage = i % kStages;
            const size_t slab = (size_t)b * a.H + h;
            const bf16* cache = reinterpret_cast<const bf16*>(a.kv) + slab * a.cap * 2 * HD + sub * 8;
            const int n = rows_to_read(len);
            for (int r = 0; r < n; ++r) {
                cp_async16(slot_addr(stage, 3 + 2 * r), cache + (size_t)r * 2 * HD);
                cp_async16(slot_addr(stage, 4 + 2 * r), cache + (size_t)r * 2 * HD + HD);
            }
        }
    };

    // lens[d] = length of the sequence of group (i + d).  A length is needed when the copies of
    // its group are issued (kDepth groups ahead) and is itself a DRAM read, so it is requested
    // kLenAhead groups before that.
    constexpr int kLenAhead = 3, kLens = kDepth + kLenAhead;
    int lens[kLens];
    pdl_launch_dependents();
    // While the kernel before this one drains, warm L2 with what the first groups will ask for.  A
    // prefetch returns nothing to the thread, so it is safe ahead of the wait: whatever the previous
    // kernel still writes reaches L2 as well, and the loads proper come after the wait.
#pragma unroll
    for (int d = 0; d < kDepth + 1; ++d) {
        const int b = seq_of(d);
        if (b >= 0) {
            const size_t slab = (size_t)b * a.H + h;
            if ((sub & 7) == 0) {  // one request per 128-byte line
                prefetch_l2(reinterpret_cast<const bf16*>(a.q) + slab * HD + sub * 8);
                if (appended) {
                    prefetch_l2(reinterpret_cast<const bf16*>(a.k_new) + slab * HD + sub * 8);
                    prefetch_l2(reinterpret_cast<const bf16*>(a.v_new) + slab * HD + sub * 8);
                }
            }
            if (within == 0) prefetch_l2(a.len + b);
        }
    }
    pdl_wait();  // nothing above read or wrote global memory
    // prologue: the first groups' q, k_new, v_new are requested before their lengths are known, so the
    // two DRAM round trips (length, then rows) overlap with them
#pragma unroll
    for (int d = 0; d < kDepth; ++d) issue_new(d);
#pragma unroll
    for (int d = 0; d < kLens; ++d) lens[d] = load_len(seq_of(d));
#pragma unroll
    for (int d = 0; d < kDepth; ++d) {
        issue_rows(d, lens[d]);
        cp_async_commit();   // group d: its rows (and, in the first group, every q, k_new, v_new above)
    }

    for (int i = 0; i < n_iter; ++i) {
        const int len_ahead = load_len(seq_of(i + kLens));
        issue_new(i + kDepth);
        issue_rows(i + kDepth, lens[kDepth]);
        cp_async_commit();
        cp_async_wait<kDepth>();  // the copies of group i have landed

        const int b = seq_of(i);
        const int len_raw = lens[0];
        const bool overflow = appended && (len_raw < 0 || len_raw + 1 > a.cap);
        const int n_old = (b >= 0 && !overflow) ? rows_to_read(len_raw) : 0;
        const int stage = i % kStages;
        const uint4* my = slots_mem + (size_t)stage * n_slots * kTokThreads + tid;
        uint4 qr = make_uint4(0, 0, 0, 0), kr = qr, vr = qr;
        if (b >= 0) {
            qr = my[0];
            if (appended) {
                kr = my[kTokThreads];
                vr = my[2 * kTokThreads];
            }
        }
        float qf[8];
        unpack8(qr, qf);
#pragma unroll
        for (int d = 0; d < 8; ++d) qf[d] *= a.scale_log2;
#if BT_TOK_X2
        const uint64_t q2[4] = {pack2(qf[0], qf[1]), pack2(qf[2], qf[3]), pack2(qf[4], qf[5]), pack2(qf[6], qf[7])};
#define TOK_DOT(r) dot8_x2(q2, r)
#else
#define TOK_DOT(r) dot8(qf, r)
#endif
        // all scores first (independent dot products and shuffles), then one max, the exponentials
        // and the weighted sum: with at most kMaxRows + 1 rows nothing needs a running rescale
        uint4 vc[kMaxRows];
        float sc[kMaxRows + 1];
#pragma unroll
        for (int r = 0; r < kMaxRows; ++r) {
            const bool v = r < n_old;
            const uint4 kc = v ? my[(size_t)(3 + 2 * r) * kTokThreads] : make_uint4(0, 0, 0, 0);
            vc[r] = v ? my[(size_t)(4 + 2 * r) * kTokThreads] : make_uint4(0, 0, 0, 0);
            const float d = row_sum<LPR>(TOK_DOT(kc));
            sc[r] = v ? d : kNegInf;
        }
        {
            const float d = row_sum<LPR>(TOK_DOT(kr));
            sc[kMaxRows] = (appended && b >= 0 && !overflow) ? d : kNegInf;
        }
#undef TOK_DOT
        float mx = sc[kMaxRows];
#pragma unroll
        for (int r = 0; r < kMaxRows; ++r) mx = fmaxf(mx, sc[r]);
        float l = 0.f, acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (mx != kNegInf) {
#if BT_TOK_X2
            uint64_t acc2[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
            for (int r = 0; r < kMaxRows; ++r) {
                const float pr = ex2(sc[r] - mx);  // 0 for masked rows
                l += pr;
                fma8_x2(acc2, pr, vc[r]);
            }
            const float pn = ex2(sc[kMaxRows] - mx);
            l += pn;
            fma8_x2(acc2, pn, vr);
#pragma unroll
            for (int i = 0; i < 4; ++i) unpack2(acc2[i], acc[2 * i], acc[2 * i + 1]);
#else
#pragma unroll
            for (int r = 0; r < kMaxRows; ++r) {
                const float pr = ex2(sc[r] - mx);  // 0 for masked rows
                l += pr;
                fma8(acc, pr, vc[r]);
            }
            const float pn = ex2(sc[kMaxRows] - mx);
            l += pn;
            fma8(acc, pn, vr);
#endif
        }
        if (b >= 0) {
            const size_t slab = (size_t)b * a.H + h;
            if (appended && !overflow) {
                bf16* cache = reinterpret_cast<bf16*>(a.kv) + slab * a.cap * 2 * HD + sub * 8;
                *reinterpret_cast<uint4*>(cache + (size_t)len_raw * 2 * HD) = kr;
                *reinterpret_cast<uint4*>(cache + (size_t)len_raw * 2 * HD + HD) = vr;
            }
            float o[8];
            const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
            for (int d = 0; d < 8; ++d) o[d] = acc[d] * inv;
            *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.out) + slab * HD + sub * 8) = pack8(o);
        }
        __syncthreads();  // all heads hold this group's (and the prefetched groups') lengths in registers
        if (b >= 0 && within == 0) {
            if (overflow)
                raise_status(a.dev_status, BT_DEV_OVERFLOW);
            else if (appended)
                a.len[b] = len_raw + 1;
            else if (n_old == 0)
                raise_status(a.dev_status, BT_DEV_EMPTY);   // a query with nothing to see: zeros out
        }
#pragma unroll
        for (int d = 0; d + 1 < kLens; ++d) lens[d] = lens[d + 1];
        lens[kLens - 1] = len_ahead;
    }
    cp_async_wait<0>();
}

#ifndef BT_TOK_DEPTH4
#define BT_TOK_DEPTH4 1
#endif
#ifndef BT_TOK_CTAS4
#define BT_TOK_CTAS4 2
#endif

template <int HD, int kDepth, int kMaxRows, int kCtasPerSm>
static cudaError_t launch_pipelined(const TokenArgs& a, int spc, int tps, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)(kDepth + 1) * (3 + 2 * kMaxRows) * kTokThreads * sizeof(uint4);
    static_assert(smem * kCtasPerSm <= 224 * 1024, "slots do not fit in shared memory");
    static PerDeviceOnce limit_raised;
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev, &sms);
    if (e != cudaSuccess) return e;
    e = raise_smem_limit_once(limit_raised, dev, token_step_pipelined_kernel<HD, kDepth, kMaxRows, kCtasPerSm>, (int)smem);
    if (e != cudaSuccess) return e;
    const int n_groups = (a.B + spc - 1) / spc;
    const int slots = sms * kCtasPerSm;
    const int grid = n_groups < slots ? n_groups : slots;
    return launch_pdl(token_step_pipelined_kernel<HD, kDepth, kMaxRows, kCtasPerSm>, dim3(grid), dim3(kTokThreads), smem, stream,
                      a, spc, tps);
}

cudaError_t launch_token_decode(const TokenArgs& a, cudaStream_t stream)
{
    const int lpr = a.hd / 8;
    const int tps = a.H * lpr;  // threads per sequence (validated <= 256 by the caller)
    // cached rows a step may have to read: all but the one being appended, or all of them when attending only
    const int max_cached = a.k_new != nullptr ? a.cap - 1 : a.cap;
    const bool attend_only_with_reset = a.k_new == nullptr && (a.reset_first || a.reset_mask != nullptr);   // general kernel
    if (a.n_q == 1 && !attend_only_with_reset && max_cached <= 12) {
        // hot path: persistent pipelined kernel; deeper pipeline when the slots are small
        int spc_p = kTokThreads / tps;
        if (spc_p > a.B) spc_p = a.B;
        if (max_cached <= 4)
            return a.hd == 64 ? launch_pipelined<64, BT_TOK_DEPTH4, 4, BT_TOK_CTAS4>(a, spc_p, tps, stream)
                              : launch_pipelined<128, BT_TOK_DEPTH4, 4, BT_TOK_CTAS4>(a, spc_p, tps, stream);
        if (max_cached <= 5)  // e.g. L_B = 4 with the paper's main prefix length P = 2: still two CTAs per SM
            return a.hd == 64 ? launch_pipelined<64, 1, 5, 2>(a, spc_p, tps, stream)
                              : launch_pipelined<128, 1, 5, 2>(a, spc_p, tps, stream);
        if (max_cached > 8)  // the longest prefixes of the prefix-length ablation (P = 8 with L_B up to 5): 9 to 12 cached rows
            return a.hd == 64 ? launch_pipelined<64, 1, 12, 1>(a, spc_p, tps, stream)
                              : launch_pipelined<128, 1, 12, 1>(a, spc_p, tps, stream);
        // Deep local caches (6 to 8 cached rows).  A batch small enough for one wave of two CTAs per SM runs
        // without a look-ahead stage (each CTA has a single group, so there is nothing to look ahead to, and
        // the halved slots let all groups be resident at once); larger ones keep one group in flight per SM.
        int dev = 0, sms = 0;
        if (current_device(&dev, &sms) == cudaSuccess && (a.B + spc_p - 1) / spc_p <= 2 * sms)
            return a.hd == 64 ? launch_pipelined<64, 0, 8, 2>(a, spc_p, tps, stream)
                              : launch_pipelined<128, 0, 8, 2>(a, spc_p, tps, stream);
        return a.hd == 64 ? launch_pipelined<64, 1, 8, 1>(a, spc_p, tps, stream)
                          : launch_pipelined<128, 1, 8, 1>(a, spc_p, tps, stream);
    }
    int spc = BT_TOK_THREADS / tps;
    if (spc < 1) spc = 1;
    if (spc > a.B) spc = a.B;
    const int threads = ((spc * tps + 31) / 32) * 32;
    const int grid = (a.B + spc - 1) / spc;
    if (a.k_new != nullptr && a.reset_first && a.reset_mask == nullptr && a.n_q <= 8 && a.n_q <= a.cap) {
        // block start: the register-resident kernel (rows kept for up to 4 or up to 8 prefix rows)
        if (a.n_q <= 4)
            return a.hd == 64 ? launch_pdl(token_block_start_kernel<64, 4>, dim3(grid), dim3(threads), 0, stream, a, spc, tps)
                              : launch_pdl(token_block_start_kernel<128, 4>, dim3(grid), dim3(threads), 0, stream, a, spc, tps);
        return a.hd == 64 ? launch_pdl(token_block_start_kernel<64, 8>, dim3(grid), dim3(threads), 0, stream, a, spc, tps)
                          : launch_pdl(token_block_start_kernel<128, 8>, dim3(grid), dim3(threads), 0, stream, a, spc, tps);
    }
    return a.hd == 64 ? launch_pdl(token_decode_kernel<64>, dim3(grid), dim3(threads), 0, stream, a, spc, tps)
                      : launch_pdl(token_decode_kernel<128>, dim3(grid), dim3(threads), 0, stream, a, spc, tps);
}

}  // namespace bt
