// Fused token-decoder step (paper section 2.4; appendix E.2): block-boundary reset, append of
// the new K,V rows to the local cache and attention confined to the current block, in one
// launch over thousands of sequences.  A group of LPR = hd/8 lanes owns one (sequence, head):
// each lane holds 16 bytes of every row, so the whole step is a handful of independent 128-bit
// loads, a few shuffles and one 128-bit store per tensor.  A CTA always covers whole sequences
// so that every head reads the old length before one thread writes the new one.
#include "bt_common.cuh"
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

template <int HD>
__global__ void __launch_bounds__(256) token_decode_kernel(TokenArgs a, int seqs_per_cta, int threads_per_seq)
{
    constexpr int LPR = RowGeo<HD>::LPR;
    const int tid = threadIdx.x;
    const int sic = tid / threads_per_seq;            // sequence within the CTA
    const int within = tid - sic * threads_per_seq;
    const int h = within / LPR, sub = within % LPR;
    const int b = blockIdx.x * seqs_per_cta + sic;
    const bool active = sic < seqs_per_cta && b < a.B;

    int len_old = 0;
    if (active) {
        const bool rst = a.reset_mask ? (a.reset_mask[b] != 0) : (a.reset_first != 0);
        len_old = rst ? 0 : a.len[b];
    }
    __syncthreads();  // every head has read len[b] before the leader overwrites it

    const bool appended = a.k_new != nullptr;
    const bool overflow = appended && (len_old < 0 || len_old + a.n_q > a.cap);
    if (len_old < 0) len_old = 0;
    if (len_old > a.cap) len_old = a.cap;

    const size_t slab = active ? (size_t)b * a.H + h : 0;
    bf16* cache = reinterpret_cast<bf16*>(a.kv) + slab * a.cap * 2 * HD + sub * 8;  // row r: K at +r*2*HD, V at +(r*2+1)*HD
    const bf16* qp = reinterpret_cast<const bf16*>(a.q) + slab * a.n_q * HD + sub * 8;
    const bf16* kp = reinterpret_cast<const bf16*>(a.k_new) + slab * a.n_q * HD + sub * 8;
    const bf16* vp = reinterpret_cast<const bf16*>(a.v_new) + slab * a.n_q * HD + sub * 8;
    bf16* op = reinterpret_cast<bf16*>(a.out) + slab * a.n_q * HD + sub * 8;

    if (a.n_q == 1 && appended) {
        // token step: the new row stays in registers, the cached rows are read once
        uint4 qr = make_uint4(0, 0, 0, 0), kr = qr, vr = qr;
        const int n_old = (active && !overflow) ? len_old : 0;
        if (active) {
            qr = ld_stream(qp);
            kr = ld_stream(kp);
            vr = ld_stream(vp);
        }
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
        // general step: n_q rows (the P prefix rows at a block start), or attend-only.
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
            const int n = (!active || overflow) ? 0 : (appended ? len_old + i + 1 : len_old);
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
            if (!appended && len_old == 0) raise_status(a.dev_status, BT_DEV_EMPTY);
        }
    }
}

cudaError_t launch_token_decode(const TokenArgs& a, cudaStream_t stream)
{
    const int lpr = a.hd / 8;
    const int tps = a.H * lpr;  // threads per sequence (validated <= 256 by the caller)
    int spc = 256 / tps;
    if (spc < 1) spc = 1;
    if (spc > a.B) spc = a.B;
    const int threads = ((spc * tps + 31) / 32) * 32;
    const int grid = (a.B + spc - 1) / spc;
    if (a.hd == 64)
        token_decode_kernel<64><<<grid, threads, 0, stream>>>(a, spc, tps);
    else
        token_decode_kernel<128><<<grid, threads, 0, stream>>>(a, spc, tps);
    return cudaGetLastError();
}

}  // namespace bt
