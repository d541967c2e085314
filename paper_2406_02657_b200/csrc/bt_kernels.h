// Internal launch interface between the C-ABI layer (bt_api.cu) and the kernels.
// Every launcher enqueues on `stream` and returns the launch's cudaError_t.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bt.h"

namespace bt {

// Everything bt_block_decode_attn checks on the host except the workspace (for the entry point that
// supplies the workspace itself and must refuse bad arguments before it enqueues anything).
bt_status validate_decode_attn_args(const bt_config* cfg, const bt_block_cache* cache, int layer, const void* q, const void* out,
                                    const uint32_t* dev_status);
// Test-only kernel behind bt_selftest_bounded_wait.
cudaError_t launch_selftest_bounded_wait(uint32_t* report, uint32_t* dev_status, cudaStream_t stream);

// Rows of a cache as the copy kernels see them: K row r of slab s at
// k + s*slab_stride + r*row_stride (elements), V likewise from v.
struct CacheView {
    void* k;
    void* v;
    int32_t* len;        // [B] for the layer
    int64_t slab_stride; // elements between consecutive (b,h) slabs
    int64_t row_stride;  // elements between consecutive rows
    int32_t cap;         // rows
};

cudaError_t launch_kv_append(const CacheView& c, int B, int H, int hd, const void* k_new, const void* v_new,
                             int n_new, uint32_t* dev_status, cudaStream_t stream);
cudaError_t launch_len_reset(int32_t* len, int B, const uint8_t* mask, cudaStream_t stream);

struct DecodeArgs {
    const void* q;       // [B][H][hd]
    void* k;             // layer base, [B][H][N_max][hd] (written only by the fused append)
    void* v;
    int32_t* len;        // [B] (written only by the fused append)
    void* out;           // [B][H][hd]
    float* ws;           // [B*H][splits][hd+4] when splits > 1
    // arrival counters, zero on entry and left zero: [B*H] (splits of a (b,h) that have written their
    // partial) then [B] (items of a sequence that are done with its length).  Needed when splits > 1 or
    // when a row is appended; may be NULL otherwise.
    int32_t* counters;
    const void* k_new;   // fused append: [B][H][hd], the row that becomes row len[b]; NULL = attention only
    const void* v_new;
    uint32_t* dev_status;
    int B, H, hd, n_max, splits;
    float scale_log2;    // softmax scale * log2(e)
};
// The streaming kernel: per-item results, or per-split partials merged by the split that finishes last.
cudaError_t launch_block_decode(const DecodeArgs& a, cudaStream_t stream);

// Decode step with m queries and m new rows per (sequence, head) (query i sees the cache and new rows 0..i).
struct MultiDecodeArgs {
    const void* q;       // [B][H][m][hd]
    const void* k_new;   // [B][H][m][hd]
    const void* v_new;
    void* k;             // layer base, [B][H][N_max][hd]
    void* v;
    int32_t* len;        // [B]
    void* out;           // [B][H][m][hd]
    int32_t* counters;   // decode workspace counters: [B*H] (unused here) then [B], zero on entry and on exit
    uint32_t* dev_status;
    int B, H, hd, n_max, m;
    float scale_log2;
};
bool multi_decode_supported(const MultiDecodeArgs& a);
cudaError_t launch_block_decode_multi(const MultiDecodeArgs& a, cudaStream_t stream);

struct TokenArgs {
    void* kv;            // layer base, [B][H][C][2][hd]
    int32_t* len;        // [B]
    const void* q;
    const void* k_new;   // may be NULL (attend only)
    const void* v_new;
    void* out;
    const uint8_t* reset_mask;
    uint32_t* dev_status;
    int B, H, hd, cap, n_q, reset_first;
    float scale_log2;
};
cudaError_t launch_token_decode(const TokenArgs& a, cudaStream_t stream);

struct PrefillArgs {
    const void* q;
    const void* k;
    const void* v;
    void* out;
    int B, H, hd, T;
    int64_t kv_seq_stride;  // rows
    float scale_log2;
};
// Plain CUDA-core kernel: any T, used for shapes the tensor-core kernel does not take.
cudaError_t launch_block_prefill_simple(const PrefillArgs& a, cudaStream_t stream);
// Tensor-core kernel (TMA + tcgen05 + TMEM): needs 16-byte aligned pointers.
bool prefill_tc_supported(const PrefillArgs& a);
cudaError_t launch_block_prefill_tc(const PrefillArgs& a, uint32_t* dev_status, cudaStream_t stream);


// y = W x + b on the tensor cores.  x [M][K], w [N][K] (row o = weights of output feature o), bias [N] or
// NULL, all bf16; fp32 accumulation, bf16 results.
//   kProjectPlain : out [M][N]
//   kProjectQkv   : M = B * n_rows rows (sequence b, row i), N = 3 * H * hd output features ordered Q, K, V,
//                   each (h, d): Q -> out [B][H][n_rows][hd]; K, V -> rows len_old[b] + i of `cache`
//                   (len_old = 0 where the reset applies); a sequence without room for n_rows rows keeps
//                   its cache.  A second launch then advances the lengths (and flags those sequences).
enum { kProjectPlain = 0, kProjectQkv = 1 };
struct ProjectArgs {
    const void* x;
    const void* w;
    const void* bias;
    void* out;
    int M, N, K;
    int mode;
    CacheView cache;          // kProjectQkv
    int n_rows, H, hd;        // kProjectQkv
    int reset_first;
    const uint8_t* reset_mask;
    uint32_t* dev_status;
};
bool project_supported(const ProjectArgs& a);
cudaError_t launch_project(const ProjectArgs& a, cudaStream_t stream);

}  // namespace bt
