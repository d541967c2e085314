/*
 * bt.h - C ABI of the Block Transformer KV-cache attention library (sm_100a).
 *
 * The library implements the attention that reads the KV cache in the Block
 * Transformer's two decoders (paper sections 2.3 and 2.4, appendix E.2):
 *   - block decoder: causal attention over a block-level KV cache with one row per
 *     L_B-token block, run once every L_B tokens (decode) or over all prompt blocks
 *     at once (prefill);
 *   - token decoder: attention confined to the current block, over a small local
 *     KV cache seeded by P prefix rows and dropped at every block boundary.
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned by the caller unless an argument
 *     is explicitly named *_host.  The library never allocates, frees or keeps
 *     device memory.
 *   - bf16 storage, fp32 arithmetic.  Outputs are bf16, rounded to nearest even
 *     from the fp32 accumulators.  Lengths are int32.
 *   - q / k_new / v_new / out tensors are contiguous [B][H][n][hd] (n = 1 may be
 *     thought of as [B][H][hd]).
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it and
 *     the call returns without synchronising.
 *   - Alignment: the kernels move data in 16-byte pieces, so every tensor pointer
 *     (q, k_new, v_new, out, the cache bases, the workspace, the staging buffers)
 *     must be 16-byte aligned and every int32 / uint32 array 4-byte aligned; a
 *     pointer that is not is refused with BT_ERR_UNSUPPORTED.
 *   - Host-detectable errors (null pointer, bad shape, unsupported head_dim, a
 *     misaligned pointer, a request larger than the capacity, workspace too small)
 *     return a non-zero bt_status before anything is enqueued: no launch, no copy,
 *     no memset.  Data-dependent conditions found on
 *     the device (a sequence whose cache is full, attention over an empty cache)
 *     never trap: the sequence is skipped or zeros are produced, and a BT_DEV_*
 *     bit is OR-ed into *dev_status (a device uint32 the caller clears and reads
 *     when it chooses; may be NULL to ignore).
 *   - softmax scale: cfg->softmax_scale, or 1/sqrt(head_dim) when it is 0 (the
 *     paper uses the Pythia / GPT-NeoX architecture and does not restate it).
 *   - Positions: the library is position-agnostic; rotary or other position
 *     encodings are applied by the caller before K is cached.
 */
#ifndef BT_H_
#define BT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BT_OK = 0,
    BT_ERR_NULL = 1,        /* a required pointer is NULL                         */
    BT_ERR_SHAPE = 2,       /* non-positive or inconsistent dimension, bad layer  */
    BT_ERR_UNSUPPORTED = 3, /* head_dim not in {64,128}, too many heads, misaligned pointer */
    BT_ERR_CAPACITY = 4,    /* n_new larger than the cache capacity               */
    BT_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than bt_workspace_bytes  */
    BT_ERR_CUDA = 6         /* a CUDA runtime call or launch failed               */
} bt_status;

/* bits of the device status word */
enum { BT_DEV_OK = 0, BT_DEV_OVERFLOW = 1, BT_DEV_EMPTY = 2, BT_DEV_TIMEOUT = 4 };

/* Problem statement in the paper's terms (section 2; model table in appendix D). */
typedef struct bt_config {
    int32_t batch;         /* B: sequences decoded together                          */
    int32_t heads;         /* H: attention heads (plain multi-head: one K,V per head) */
    int32_t head_dim;      /* hd: 64 or 128                                          */
    int32_t block_len;     /* L_B: tokens per block, >= 1                            */
    int32_t prefix_len;    /* P: prefix rows projected from the context embedding    */
    int32_t max_blocks;    /* N_max: block-cache capacity in rows (= blocks)         */
    int32_t n_layers;      /* caches and length arrays hold this many layers         */
    int32_t decode_splits; /* 0: library chooses how many ways bt_block_decode_attn
                              splits the row range; >0: forced (tests, tuning)       */
    float softmax_scale;   /* 0 => 1/sqrt(head_dim)                                  */
    int32_t prefill_plain; /* non-zero: bt_block_prefill_attn uses its CUDA-core kernel
                              instead of the tensor-core one (testing; odd alignments) */
} bt_config;

/* Block-level KV cache (section 2.3): one row per block.
 *   k, v : bf16 [n_layers][B][H][N_max][hd]
 *   len  : int32 [n_layers][B]   rows valid per (layer, sequence)                   */
typedef struct bt_block_cache {
    void* k;
    void* v;
    int32_t* len;
} bt_block_cache;

/* Local KV cache of the token decoder (section 2.4): capacity C = P + L_B rows, K and V
 * rows interleaved so that one (sequence, head) is one contiguous run.
 *   kv  : bf16 [n_layers][B][H][C][2][hd]   ([..][c][0][:] = K row c, [..][c][1][:] = V row c)
 *   len : int32 [n_layers][B]                                                       */
typedef struct bt_local_cache {
    void* kv;
    int32_t* len;
} bt_local_cache;

/* Library version (major*10000 + minor*100 + patch) and a printable status name. */
int bt_version(void);
const char* bt_status_string(bt_status s);

/* Number of ways the block-decoder decode kernel splits each (sequence, head) row range for this
 * config (>= 1), and the size of the workspace of the decode calls: splits * B * H * (hd + 4) floats
 * of per-split partial results when splits > 1, then B * H + B int32 arrival counters.  Both
 * return 0 on an invalid config.
 *
 * bt_workspace_init zeroes the counters (asynchronously, on the stream).  A workspace must be
 * initialised once - by this call, or by zero-filling it - before its first use; every decode
 * call leaves the counters at zero again, so it is never needed a second time, except after a
 * call that raised BT_DEV_TIMEOUT (which may leave counts behind).  The partial results need no
 * initialisation.  A workspace serves one call at a time: calls that can overlap on the GPU need
 * one each.                                                                                   */
int bt_decode_splits(const bt_config* cfg);
size_t bt_workspace_bytes(const bt_config* cfg);
bt_status bt_workspace_init(const bt_config* cfg, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Block-decoder KV append (sections 2.1 and 2.3: the K,V of every processed block are cached,
 * one row per block, written once every L_B tokens; n_new = T writes a whole prefilled prompt).
 * For each sequence b: rows len[b] .. len[b]+n_new-1 of every head receive k_new / v_new
 * [B][H][n_new][hd], then len[b] += n_new.  A sequence with len[b] + n_new > N_max is left
 * untouched and BT_DEV_OVERFLOW is raised.  Returns BT_ERR_CAPACITY if n_new > N_max.
 */
bt_status bt_block_kv_append(const bt_config* cfg, bt_block_cache* cache, int layer,
                             const void* k_new, const void* v_new, int n_new,
                             uint32_t* dev_status, void* stream);

/*
 * Block-decoder decode attention (section 2.3; appendix E.2 "decode IO"): for each (b,h),
 *   out[b,h,:] = sum_j softmax_j(scale * q[b,h,:] . K[b,h,j,:]) * V[b,h,j,:],  j < len[b],
 * i.e. the query of the newest block attends to every cached block including its own row
 * len[b]-1.  q, out: [B][H][hd].  len[b] == 0 gives zeros and BT_DEV_EMPTY.
 * workspace: device scratch of at least bt_workspace_bytes(cfg) bytes, initialised as described
 * there (may be NULL when bt_decode_splits(cfg) is 1: an unsplit row range needs none).  With a
 * split range each part writes its partial result there and the part that finishes last combines
 * them by the log-sum-exp rule, inside the same launch.
 */
bt_status bt_block_decode_attn(const bt_config* cfg, const bt_block_cache* cache, int layer,
                               const void* q, void* out, void* workspace, size_t workspace_bytes,
                               uint32_t* dev_status, void* stream);

/*
 * One block-decoder decode step of a layer in a single launch (section 2.3: per generated block,
 * the block's K,V are cached and its query attends to every cached block including itself):
 * exactly bt_block_kv_append with n_new = 1 followed by bt_block_decode_attn.  For each sequence
 * b with len[b] < N_max: row len[b] of every head receives k_new / v_new [B][H][hd], the query
 * attends to rows 0 .. len[b] (the new row comes from k_new / v_new, the rest from the cache), and
 * len[b] += 1.  A sequence whose cache is full is left as it is, attended over its N_max rows, and
 * BT_DEV_OVERFLOW is raised.  workspace: required (never NULL), as for bt_block_decode_attn.
 * The cache rows, the lengths and out are all written by this one launch; k_new, v_new and q must
 * not alias them.
 */
bt_status bt_block_decode_step(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q,
                               const void* k_new, const void* v_new, void* out, void* workspace,
                               size_t workspace_bytes, uint32_t* dev_status, void* stream);

/*
 * Decode step of the "densified" block decoder the paper proposes as future work (appendix
 * "Discussion and future works": a block is represented by L_B sub-block tokens instead of one, so
 * a step appends L_B rows and runs L_B queries while the cache is fetched once).  For each
 * sequence b with len[b] + n_q <= N_max: rows len[b] .. len[b]+n_q-1 of every head receive
 * k_new / v_new [B][H][n_q][hd]; query i of q [B][H][n_q][hd] attends to rows 0 .. len[b]+i
 * (every cached row and the new rows 0..i); out [B][H][n_q][hd]; len[b] += n_q.  A sequence
 * without room for all n_q rows is left as it is, every query attends over its len[b] rows, and
 * BT_DEV_OVERFLOW is raised.  n_q = 1 computes what bt_block_decode_step computes.
 * Scores and weighted sums run on the tensor cores (bf16 inputs, fp32 accumulation; the softmax
 * weights are rounded to bf16 where they meet V).  Supported: 1 <= n_q <= 8, N_max >= 32, all
 * pointers 16-byte aligned; otherwise BT_ERR_UNSUPPORTED.  The row range is
 * never split.  workspace: required, as for bt_block_decode_step.
 */
bt_status bt_block_decode_step_multi(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q,
                                     const void* k_new, const void* v_new, int n_q, void* out,
                                     void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                     void* stream);

/*
 * bt_block_decode_attn for callers that cannot supply a workspace.  (The paper has no
 * counterpart: this is a property of the library, not of the method.)  It computes exactly what
 * bt_block_decode_attn computes, with the per-split partials kept in a fixed array inside the
 * loaded library instead of caller memory.  It is meant for hosts that have no device memory
 * left to give (a serving process whose pool took the whole GPU at start-up) or that must not
 * allocate where they call from (cudaMalloc synchronises the whole device, which a decode loop
 * with a latency budget cannot accept).  Neither this call nor anything it reaches allocates or
 * frees device memory.
 *   - Limit: bt_workspace_bytes(cfg) must not exceed BT_STATIC_WORKSPACE_BYTES, else
 *     BT_ERR_WORKSPACE is returned.  Like every refused call, one refused here has enqueued
 *     nothing and has not touched the shared array.  Every GPU on which the library is
 *     loaded holds that many bytes until the process exits.
 *   - The first call on each device whose config splits the row range looks up the array's
 *     address on that device (the device must be current, as for every call here, and own the
 *     buffers passed in).  Make that first call outside any stream capture.
 *   - All calls on one device share the array, whatever their config.  The caller never clears
 *     it: each call zeroes its own arrival counters first (a memset on the stream), and every
 *     partial is written before it is read within one call.  But
 *     two calls that can overlap on the GPU (different streams, no dependency) race on it:
 *     order them, or give one of them bt_block_decode_attn with its own workspace.
 * Other arguments, results and errors are those of bt_block_decode_attn.
 */
#define BT_STATIC_WORKSPACE_BYTES (2u << 20) /* 2 MiB */
bt_status bt_block_decode_attn_noalloc(const bt_config* cfg, const bt_block_cache* cache, int layer,
                                       const void* q, void* out, uint32_t* dev_status, void* stream);

/*
 * Block boundary of the token decoder (Figure 1; section 2.4): the local K,V of a finished
 * block are never read again, so the cache is dropped by zeroing its length; no data is
 * cleared.  seq_mask: NULL resets every sequence, else uint8 [B], non-zero = reset.
 */
bt_status bt_local_kv_reset(const bt_config* cfg, bt_local_cache* cache, int layer,
                            const uint8_t* seq_mask, void* stream);

/*
 * Append n_new rows to the local cache without attending (section 2.4: prefix rows, or the
 * partially filled most recent prompt block, the only prompt tokens the token decoder sees).
 * Same semantics as bt_block_kv_append with capacity C = P + L_B.
 */
bt_status bt_local_kv_append(const bt_config* cfg, bt_local_cache* cache, int layer,
                             const void* k_new, const void* v_new, int n_new,
                             uint32_t* dev_status, void* stream);

/*
 * Fused token-decoder step (section 2.4; appendix E.2): in one launch, per sequence b,
 *   1. reset:  if reset_mask ? reset_mask[b] : reset_first, then len[b] = 0 (block boundary);
 *   2. append: rows len[b] .. len[b]+n_q-1 receive k_new / v_new [B][H][n_q][hd];
 *   3. attend: new row i (i < n_q) attends to local rows 0 .. len_old+i, i.e. the prefix rows,
 *      the earlier tokens of the same block and itself - never anything outside the block;
 *   4. len[b] += n_q.
 * n_q = 1 for a token step; n_q = P at a block start appends the P prefix rows, causally
 * masked among themselves.  k_new == v_new == NULL: nothing is appended (the rows were cached
 * by bt_local_qkv_project_append); the n_q queries are those of the last n_q cached rows, so
 * query i attends to rows 0 .. len[b]-n_q+i - with n_q = 1, rows 0 .. len[b]-1 (zeros and
 * BT_DEV_EMPTY for a query with no row to see).
 * A sequence without room for n_q rows is skipped: nothing written, zeros out,
 * BT_DEV_OVERFLOW.  q, out: [B][H][n_q][hd].
 */
bt_status bt_token_decode_attn(const bt_config* cfg, bt_local_cache* cache, int layer,
                               const void* q, const void* k_new, const void* v_new, int n_q,
                               int reset_first, const uint8_t* reset_mask, void* out,
                               uint32_t* dev_status, void* stream);

/*
 * Block-decoder prefill attention (sections 2.1 and 2.3: the prefill stage processes all
 * prompt positions in parallel; the block decoder does so over T = L / L_B blocks):
 *   out[b,h,t,:] = sum_{j<=t} softmax_j(scale * q[b,h,t,:] . k[b,h,j,:]) * v[b,h,j,:],  t < T.
 * q, out: [B][H][T][hd].  k, v: rows hd apart; (b,h) slab s starts s * kv_seq_stride rows
 * after the base, so kv_seq_stride = T for packed tensors and = N_max when k, v point at a
 * layer of a block cache that already holds the prompt's rows.  Requires kv_seq_stride >= T.
 * Runs on the tensor cores (TMA-fed tcgen05 MMA, accumulators in tensor memory), or, when
 * cfg->prefill_plain is set, on a CUDA-core kernel (an order of magnitude slower; a cross-check).
 * The library never switches between the two on its own.  Every wait inside the tensor-core
 * kernel is bounded; one that runs out raises BT_DEV_TIMEOUT in *dev_status and leaves the
 * affected output rows unwritten.
 */
bt_status bt_block_prefill_attn(const bt_config* cfg, const void* q, const void* k, const void* v,
                                int n_blocks, int64_t kv_seq_stride, void* out, uint32_t* dev_status,
                                void* stream);

/*
 * One block-decoder decode step of one layer driven from HOST buffers (bt_block_decode_step with
 * the copies around it, section 2.3): q_host, k_new_host,
 * v_new_host [B][H][hd] bf16 are copied to the caller's device staging buffers q_dev, k_dev,
 * v_dev, the row is appended and attended over in one launch, and out_dev is copied to out_host [B][H][hd].
 * Host buffers should be pinned; all copies are asynchronous on `stream`.
 */
bt_status bt_block_decode_step_host(const bt_config* cfg, bt_block_cache* cache, int layer,
                                    const void* q_host, const void* k_new_host, const void* v_new_host,
                                    void* out_host, void* q_dev, void* k_dev, void* v_dev, void* out_dev,
                                    void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                    void* stream);

/*
 * Prefix projection (section 2.4; appendix on token-decoder variants, "Prefix"): the context embedding
 * the block decoder produced for a block is projected into the P = cfg->prefix_len prefix token
 * embeddings that seed the token decoder:
 *   prefix_out[b][p][:] = W_p ctx[b][:] + bias_p,   p < P.
 * ctx: bf16 [B][D], D = H * hd.  w_prefix: bf16 [P*D][D], row p*D + d holds the weights of dimension d
 * of prefix token p.  bias: bf16 [P*D] or NULL.  prefix_out: bf16 [B][P][D].  A dense product on the
 * tensor cores (TMA-fed tcgen05 MMA, fp32 accumulation in tensor memory), results rounded to bf16.
 * dev_status: BT_DEV_TIMEOUT if a (bounded) wait inside the kernel ran out.
 */
bt_status bt_prefix_project(const bt_config* cfg, const void* ctx, const void* w_prefix, const void* bias,
                            void* prefix_out, uint32_t* dev_status, void* stream);

/*
 * QKV projection whose K and V go straight into the cache (sections 2.1 and 2.3: the K,V of every
 * processed block are cached; section 2.4: likewise the rows of the current block, locally), so that
 * no separate append pass reads and writes them again.  x: bf16 [B][n_rows][D], the layer's input for
 * the n_rows new positions of every sequence (one block embedding; P prefix embeddings; one token).
 * w_qkv: bf16 [3*D][D], output features ordered Q, K, V and (head, dim) inside each; bias: bf16 [3*D]
 * or NULL.  With y = w_qkv x + bias per row (fp32 accumulation, rounded to bf16):
 *   q_out[b][h][i][:] = the Q part of row i              (bf16 [B][H][n_rows][hd], the layout the
 *                                                         attention calls take)
 *   cache rows len[b]+i of head h = the K and V parts,   i < n_rows
 *   len[b] += n_rows.
 * A sequence without room for n_rows more rows keeps its cache and length, BT_DEV_OVERFLOW is raised
 * (its q_out rows are still written).  Two launches: the product with the cache-writing epilogue, then
 * a small one that advances the lengths once every tile has read the old ones.
 * Attention then runs over the cache as it stands: bt_block_decode_attn for the block decoder,
 * bt_token_decode_attn with k_new = v_new = NULL (n_q = n_rows) for the token decoder.
 * Returns BT_ERR_CAPACITY if n_rows exceeds the cache capacity.
 *
 * The local form adds the block-boundary reset of bt_token_decode_attn: where
 * (reset_mask ? reset_mask[b] : reset_first) holds, sequence b's rows land at index 0 .. n_rows-1
 * and its length becomes n_rows.
 */
bt_status bt_block_qkv_project_append(const bt_config* cfg, bt_block_cache* cache, int layer, const void* x,
                                      int n_rows, const void* w_qkv, const void* bias, void* q_out,
                                      uint32_t* dev_status, void* stream);
bt_status bt_local_qkv_project_append(const bt_config* cfg, bt_local_cache* cache, int layer, const void* x,
                                      int n_rows, const void* w_qkv, const void* bias, int reset_first,
                                      const uint8_t* reset_mask, void* q_out, uint32_t* dev_status, void* stream);

/*
 * Self-test of the bounded waits (test support; the paper has no counterpart).  Every wait inside the
 * library's kernels is on a shared-memory barrier and is bounded - by a poll count in the streaming
 * decode kernels, by wall time in the prefill kernel - and raises BT_DEV_TIMEOUT when the bound runs
 * out.  This call launches one small CTA that runs those same two wait routines, with short limits
 * (a few thousand polls; 0.2 ms), on barriers that nothing will ever complete, plus a control wait on
 * a completed barrier.  No copy is issued, so nothing is in flight when the waits give up; the kernel
 * ends normally and the context stays usable.
 *   report     : optional device uint32[4]: [0] the poll-bounded wait gave up (1 expected),
 *                [1] the time-bounded wait gave up (1 expected), [2] the control wait succeeded
 *                (1 expected), [3] nanoseconds the time-bounded wait took.
 *   dev_status : required; BT_DEV_TIMEOUT is OR-ed in when a wait gave up.
 */
bt_status bt_selftest_bounded_wait(uint32_t* report, uint32_t* dev_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BT_H_ */
