/*
 * CPU oracle for the Block Transformer's KV-cache attention path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * CUDA library must compute.  It shares no code, header, table or helper with the
 * CUDA path, and the product never calls it: only the tests, the smoke check and
 * the benchmark's cpu_baseline / reference legs do.
 *
 * What it states (paper section 2.1 "primer", sections 2.3 and 2.4, appendix E.2):
 *   - a KV cache is an array of rows plus an integer length; caching changes cost,
 *     not the function computed;
 *   - the block decoder is an ordinary causal transformer over blocks: the query
 *     of block i sees cache rows 0..i (its own row included);
 *   - the token decoder attends only inside the current block: to the P prefix
 *     rows projected from the context embedding and to the tokens of the same
 *     block decoded so far; its cache is dropped at each block boundary;
 *   - attention itself is softmax(scale * q.K^T) V, written here as the textbook
 *     two-pass formula: scores, max, exponentials, sums, divide.  No tiling, no
 *     running rescale, no splitting of the row range;
 *   - the linear maps either side of that path (section 2.4 and the appendix on
 *     token-decoder variants: the context embedding is projected into P prefix token
 *     embeddings; sections 2.1 and 2.3: each layer caches the K,V it computes from
 *     its input) are y = W x + b as a triple loop, and "project, then cache" is that
 *     product followed by the ordinary append.
 *
 * Precision: the file is compiled twice.  REAL=double gives the primary oracle
 * (symbols bto_*), REAL=float gives a single-precision twin (bto_*_f32) used to
 * check that the result does not hinge on the precision of the reference.
 * bf16 inputs arrive as uint16 bit patterns and are widened exactly.
 * Outputs stay in REAL (never rounded to bf16) so that a comparison sees the
 * rounding of the implementation under test.
 *
 * Pins (tests/test_oracle_*.py): closed forms (one row -> that row's V; equal
 * keys or q = 0 -> mean of V; one dominant key -> its V), rows of softmax sum to
 * one, convex-hull bound, permutation invariance, a brute-force restatement in
 * pure Python on tiny inputs, the library routine for scaled-dot-product
 * attention in float64, L_B = 1 equals vanilla causal attention, cached decode
 * equals the matching row of the full recompute, no dependence on other blocks,
 * the integer schedule model, and planted-mistake tests.  The projections: identity
 * and one-hot weights give back rows of the input bit for bit, numpy's float64
 * matrix product, zero input gives the bias, and "project-then-append" equals
 * kv_append of separately projected, separately rounded rows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef REAL
#define REAL double
#endif
#ifndef SUFFIX
#define SUFFIX
#endif
#define CAT_(a, b) a##b
#define CAT(a, b) CAT_(a, b)
#define FN(name) CAT(name, SUFFIX)

/* bits of the status word the append/attend steps may raise (same meaning as the
 * library's device status word, restated here, not included from it) */
#define ST_OVERFLOW 1u
#define ST_EMPTY 2u

static inline REAL widen(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (REAL)f;
}

static inline REAL real_exp(REAL x) { return sizeof(REAL) == sizeof(float) ? (REAL)expf((float)x) : (REAL)exp((double)x); }

/*
 * Softmax attention of one query over n rows (section 2.1: every decoding step
 * attends to the cached K,V of all allowed preceding positions).
 *   s_j = scale * sum_d q_d K[j][d];  p_j = exp(s_j - max s) / sum_j exp(s_j - max s)
 *   out_d = sum_j p_j V[j][d]
 * K and V rows are hd apart.  If probs != NULL the n probabilities are stored too.
 * n == 0 gives zeros.
 */
static void attend_rows(const uint16_t* q, const uint16_t* K, const uint16_t* V, int n, int hd,
                        REAL scale, REAL* out, REAL* probs)
{
    for (int d = 0; d < hd; ++d) out[d] = 0;
    if (n <= 0) return;
    REAL* s = (REAL*)malloc(sizeof(REAL) * (size_t)n);
    REAL mx = 0;
    for (int j = 0; j < n; ++j) {
        REAL acc = 0;
        for (int d = 0; d < hd; ++d) acc += widen(q[d]) * widen(K[(size_t)j * hd + d]);
        s[j] = scale * acc;
        if (j == 0 || s[j] > mx) mx = s[j];
    }
    REAL denom = 0;
    for (int j = 0; j < n; ++j) {
        s[j] = real_exp(s[j] - mx);
        denom += s[j];
    }
    for (int j = 0; j < n; ++j) {
        REAL p = s[j] / denom;
        if (probs) probs[j] = p;
        for (int d = 0; d < hd; ++d) out[d] += p * widen(V[(size_t)j * hd + d]);
    }
    free(s);
}

/* Exposed for the "rows sum to one" and closed-form pins. */
void FN(bto_attend)(const uint16_t* q, const uint16_t* K, const uint16_t* V, int n, int hd,
                    double scale, REAL* out, REAL* probs)
{
    attend_rows(q, K, V, n, hd, (REAL)scale, out, probs);
}

/*
 * Append n_new rows to a cache [B][H][cap][hd] (section 2.1: the K,V of processed
 * positions are kept so later steps can attend to them).  Rows go to indices
 * len[b] .. len[b]+n_new-1, then len[b] += n_new.  A sequence without room is left
 * untouched and ST_OVERFLOW is raised.  Used for the block cache (section 2.3,
 * one row per block) and the local cache (section 2.4, capacity P + L_B).
 * k_new, v_new: [B][H][n_new][hd].
 */
void FN(bto_kv_append)(int B, int H, int hd, int cap, uint16_t* kc, uint16_t* vc, int32_t* len,
                       const uint16_t* k_new, const uint16_t* v_new, int n_new, uint32_t* status)
{
    for (int b = 0; b < B; ++b) {
        if (len[b] < 0 || len[b] + n_new > cap) {
            *status |= ST_OVERFLOW;
            continue;
        }
        for (int h = 0; h < H; ++h)
            for (int i = 0; i < n_new; ++i) {
                size_t dst = (((size_t)b * H + h) * cap + (size_t)(len[b] + i)) * hd;
                size_t src = (((size_t)b * H + h) * n_new + (size_t)i) * hd;
                memcpy(kc + dst, k_new + src, sizeof(uint16_t) * (size_t)hd);
                memcpy(vc + dst, v_new + src, sizeof(uint16_t) * (size_t)hd);
            }
        len[b] += n_new;
    }
}

/*
 * Block-decoder decode attention (section 2.3): one query per (sequence, head)
 * over cache rows 0..len[b]-1; the row appended for the current block is row
 * len[b]-1, so a block attends to itself.  q: [B][H][hd]; out: [B][H][hd].
 * An empty cache gives zeros and ST_EMPTY.
 */
void FN(bto_block_decode_attn)(int B, int H, int hd, int cap, const uint16_t* kc, const uint16_t* vc,
                               const int32_t* len, const uint16_t* q, double scale, REAL* out,
                               uint32_t* status)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            size_t bh = (size_t)b * H + h;
            int n = len[b];
            if (n <= 0) {
#pragma omp atomic
                *status |= ST_EMPTY;
                n = 0;
            }
            attend_rows(q + bh * hd, kc + bh * cap * hd, vc + bh * cap * hd, n, hd, (REAL)scale,
                        out + bh * hd, NULL);
        }
}

/*
 * Block boundary (Figure 1 caption, section 2.4): the K,V of a finished block are
 * never read again, so the local cache is dropped by setting its length to zero.
 * mask == NULL resets every sequence, otherwise those with mask[b] != 0.
 */
void FN(bto_local_kv_reset)(int B, int32_t* len, const uint8_t* mask)
{
    for (int b = 0; b < B; ++b)
        if (!mask || mask[b]) len[b] = 0;
}

/*
 * Token-decoder step (section 2.4, appendix E.2): optionally reset at a block
 * boundary, append the n_q new rows, and let new row i (i < n_q) attend to local
 * rows 0..len_old+i: the prefix rows, the earlier tokens of the same block, and
 * itself.  Nothing outside the block is visible.  n_q = 1 for a token step;
 * n_q = P at a block start appends the prefix rows with a causal mask among them
 * (the token decoder is an autoregressive transformer).
 * With k_new == NULL nothing is appended: the n_q queries are those of the last
 * n_q rows already in the cache (written there by the projection that cached
 * them), so query i attends to rows 0..len-n_q+i - the same causal rule, counted
 * from the end; n_q = 1 attends to rows 0..len-1.
 * q, k_new, v_new: [B][H][n_q][hd]; out: [B][H][n_q][hd]; cache [B][H][cap][hd].
 * Overflow: sequence skipped (no write, zeros out, ST_OVERFLOW).  Attend-only on
 * an empty cache: zeros and ST_EMPTY.
 */
void FN(bto_token_decode_attn)(int B, int H, int hd, int cap, uint16_t* kc, uint16_t* vc, int32_t* len,
                               const uint16_t* q, const uint16_t* k_new, const uint16_t* v_new,
                               int n_q, int reset_first, const uint8_t* reset_mask, double scale,
                               REAL* out, uint32_t* status)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        uint32_t st = 0;
        int do_reset = reset_mask ? (reset_mask[b] != 0) : (reset_first != 0);
        if (do_reset) len[b] = 0;
        int len_old = len[b];
        int appended = (k_new != NULL);
        if (appended && (len_old < 0 || len_old + n_q > cap)) {
            st |= ST_OVERFLOW;
            for (int h = 0; h < H; ++h)
                for (int i = 0; i < n_q; ++i)
                    for (int d = 0; d < hd; ++d) out[((((size_t)b * H + h) * n_q) + i) * hd + d] = 0;
        } else {
            for (int h = 0; h < H; ++h) {
                size_t bh = (size_t)b * H + h;
                uint16_t* Kb = kc + bh * cap * hd;
                uint16_t* Vb = vc + bh * cap * hd;
                if (appended)
                    for (int i = 0; i < n_q; ++i) {
                        memcpy(Kb + (size_t)(len_old + i) * hd, k_new + (bh * n_q + i) * hd, sizeof(uint16_t) * (size_t)hd);
                        memcpy(Vb + (size_t)(len_old + i) * hd, v_new + (bh * n_q + i) * hd, sizeof(uint16_t) * (size_t)hd);
                    }
                for (int i = 0; i < n_q; ++i) {
                    int n = appended ? len_old + i + 1 : len_old - n_q + i + 1;
                    if (n <= 0) st |= ST_EMPTY;
                    attend_rows(q + (bh * n_q + i) * hd, Kb, Vb, n, hd, (REAL)scale, out + (bh * n_q + i) * hd, NULL);
                }
            }
            if (appended) len[b] = len_old + n_q;
        }
        if (st) {
#pragma omp atomic
            *status |= st;
        }
    }
}

/*
 * Block-decoder prefill (sections 2.1 and 2.3): dense causal attention over the T
 * prompt blocks; query block t sees blocks 0..t.  q, out: [B][H][T][hd];
 * k, v: rows hd apart, consecutive (b,h) slabs kv_seq_stride rows apart (T when
 * packed, the cache capacity when k, v point into a block cache).
 */
void FN(bto_block_prefill_attn)(int B, int H, int T, int hd, const uint16_t* q, const uint16_t* k,
                                const uint16_t* v, long long kv_seq_stride, double scale, REAL* out)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh)
        for (int t = 0; t < T; ++t) {
            const uint16_t* Kb = k + (size_t)bh * (size_t)kv_seq_stride * hd;
            const uint16_t* Vb = v + (size_t)bh * (size_t)kv_seq_stride * hd;
            attend_rows(q + ((size_t)bh * T + t) * hd, Kb, Vb, t + 1, hd, (REAL)scale,
                        out + ((size_t)bh * T + t) * hd, NULL);
        }
}

/*
 * Linear map y = W x + b over M rows (the appendix on token-decoder variants, "Prefix": the
 * context embedding is projected into prefix token embeddings; any nn.Linear-shaped layer).
 * x: [M][K] bf16 bits; W: [N][K] bf16 bits (row o holds the weights of output feature o);
 * bias: [N] bf16 bits or NULL; y: [M][N] REAL, not rounded.
 */
void FN(bto_linear)(int M, int K, int N, const uint16_t* x, const uint16_t* W, const uint16_t* bias, REAL* y)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int o = 0; o < N; ++o) {
            REAL acc = bias ? widen(bias[o]) : (REAL)0;
            for (int k = 0; k < K; ++k) acc += widen(x[(size_t)m * K + k]) * widen(W[(size_t)o * K + k]);
            y[(size_t)m * N + o] = acc;
        }
}

/* Nearest bf16 (ties to even) of a finite REAL, as bits; bf16 keeps 8 significant bits. */
static uint16_t round_to_bf16(REAL v)
{
    double a = fabs((double)v);
    if (a == 0) return signbit((double)v) ? 0x8000u : 0;
    int e = ilogb(a);                     /* 2^e <= a < 2^(e+1) */
    if (e < -126) e = -126;               /* subnormal range: fixed spacing */
    double q = nearbyint(ldexp(a, 7 - e)); /* default rounding mode: ties to even */
    float f = (float)ldexp(q, e - 7);     /* exactly representable */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)((u >> 16) | (signbit((double)v) ? 0x8000u : 0));
}
uint16_t FN(bto_round_to_bf16)(double v) { return round_to_bf16((REAL)v); }

/*
 * QKV projection whose K,V go straight into a cache (sections 2.1 and 2.3: the K,V of every
 * processed block are cached; section 2.4: likewise for the rows of the current block in the
 * local cache).  x: [B][n][D] bf16 bits, D = H*hd; W: [3D][D] with output features ordered
 * Q (h*hd+d), then K, then V; bias [3D] or NULL.
 *   y = W x + b  per row;  q_out[b][h][i][d] = y_Q (REAL, not rounded);
 *   the K and V parts, rounded to bf16 (the cache's storage type), are appended to sequence b's
 *   cache at rows len[b]..len[b]+n-1 exactly as bto_kv_append does, after the optional reset
 *   (reset_mask ? reset_mask[b] : reset_first) that bto_token_decode_attn also knows.
 * A sequence without room keeps its cache and length (ST_OVERFLOW); its q is still produced.
 */
void FN(bto_qkv_project_append)(int B, int n, int H, int hd, int cap, const uint16_t* x, const uint16_t* W,
                                const uint16_t* bias, uint16_t* kc, uint16_t* vc, int32_t* len, int reset_first,
                                const uint8_t* reset_mask, REAL* q_out, uint32_t* status)
{
    const int D = H * hd;
    REAL* y = (REAL*)malloc(sizeof(REAL) * (size_t)B * n * 3 * D);
    FN(bto_linear)(B * n, D, 3 * D, x, W, bias, y);
    uint16_t* k_new = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)B * n * D);
    uint16_t* v_new = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)B * n * D);
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < n; ++i)
            for (int h = 0; h < H; ++h)
                for (int d = 0; d < hd; ++d) {
                    const REAL* row = y + ((size_t)b * n + i) * 3 * D;
                    size_t o = ((((size_t)b * H + h) * n) + i) * hd + d;   /* [B][H][n][hd] */
                    q_out[o] = row[h * hd + d];
                    k_new[o] = round_to_bf16(row[D + h * hd + d]);
                    v_new[o] = round_to_bf16(row[2 * D + h * hd + d]);
                }
    for (int b = 0; b < B; ++b)
        if (reset_mask ? (reset_mask[b] != 0) : (reset_first != 0)) len[b] = 0;
    FN(bto_kv_append)(B, H, hd, cap, kc, vc, len, k_new, v_new, n, status);
    free(y);
    free(k_new);
    free(v_new);
}
