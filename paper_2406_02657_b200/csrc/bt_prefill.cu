// Block-decoder prefill attention on the 5th-generation tensor cores (paper sections 2.1, 2.3:
// the prefill stage processes all prompt blocks in parallel; causal over blocks).
//
// One CTA owns 128 query blocks of one (sequence, head) and walks the key/value blocks
// 0 .. diagonal in tiles of 128; two CTAs share an SM (96 KB of shared memory and 256 tensor-
// memory columns each), so one CTA's softmax overlaps the other's MMAs and loads:
//   warp 4 (one lane): TMA producer and tcgen05.mma issuer - Q once, then per tile S = Q K^T into
//                      tensor memory and O += P V with P read from tensor memory (the probabilities
//                      never visit shared memory); K_j+1 is requested as soon as S_j has consumed
//                      K_j, V_j+1 as soon as P_j V_j has consumed V_j
//   warps 0-3        : softmax - each thread owns one query row (= one TMEM lane) and holds its
//                      128 scores in registers: one batch of tensor-memory loads, row maximum,
//                      exp2 (packed fp32x2 multiply-adds around it), bf16 P written over the S
//                      columns, running row sum; on the diagonal tile a warp skips the column
//                      chunks that are masked for all of its rows.  O is rescaled in TMEM only when
//                      the row maximum grew by more than 2^8 (otherwise the old reference is kept,
//                      exact because O and the row sum share it)
// All waits are bounded: a wait that runs out raises BT_DEV_TIMEOUT and the CTA winds down.
#include <cuda.h>

#include "bt_common.cuh"
#include "bt_kernels.h"

namespace bt {
namespace pf {

constexpr int BM = 128;             // query rows per CTA
constexpr int BN = 128;             // key/value rows per tile
constexpr int kBoxBytes = 128 * 128;  // one TMA box: 128 rows x 64 bf16 (128 bytes, swizzled)
constexpr int kThreads = 160;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

// ---- barrier slots in shared memory
enum { B_QFULL = 0, B_KFULL, B_VFULL, B_KEMPTY, B_VEMPTY, B_SFULL, B_PFULL, B_OFULL, B_COUNT };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* dev_status)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    raise_status(dev_status, BT_DEV_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
          "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
          "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
          "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}

struct Params {
    void* out;
    uint32_t* dev_status;
    int T, n_qtiles;
    float scale_log2;
};

// 16 consecutive 32-bit columns of this thread's TMEM lane (32 packed bf16).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]: A (the bf16 probabilities) is read from tensor memory.
__device__ __forceinline__ void mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Issue (without waiting) the load of 32 consecutive 32-bit columns of this thread's TMEM lane
// into r[0..31].  The registers hold the data only after tmem_ld_fence32 on the same registers.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// Placed after tmem_wait_ld(): makes every later use of r[0..31] depend on a statement that follows
// the wait, so no consumer can be scheduled ahead of it.  Emits no instruction.
__device__ __forceinline__ void tmem_ld_fence32(uint32_t* r)
{
    asm volatile(""
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}
__device__ __forceinline__ void tmem_st16p(uint32_t taddr, const uint32_t* v)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}

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

template <int HD>
constexpr int smem_bytes()
{
    // Q, K, V tiles (HD/64 boxes each) + barriers, plus 1024 to align
    return 1024 + (HD / 64) * kBoxBytes * 3 + 256;
}

constexpr uint32_t kTmemCols = 256;  // S/P: 128 columns, O: up to 128 columns; two CTAs fit in the SM's 512

template <int HD>
__global__ void __launch_bounds__(kThreads, 2)
block_prefill_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        const __grid_constant__ CUtensorMap mapV, Params p)
{
    constexpr int NB = HD / 64;                 // TMA boxes per operand tile
    constexpr uint32_t TILE_BYTES = NB * kBoxBytes;
    constexpr uint32_t IDESC_S = make_idesc(BM, BN, false);
    constexpr uint32_t IDESC_O = make_idesc(BM, HD, true);
    constexpr uint32_t COL_S = 0, COL_O = BN;   // TMEM columns: S (fp32) / P (bf16 pairs, in place) | O

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sQ = base;
    const uint32_t sK = sQ + TILE_BYTES;
    const uint32_t sV = sK + TILE_BYTES;
    const uint32_t sBar = sV + TILE_BYTES;      // B_COUNT x 8 bytes
    uint8_t* gen_tail = gen_base + (sBar - base);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_tail + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_tail + B_COUNT * 8 + 8);
    auto bar = [&](int i) { return sBar + 8u * i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.x / p.n_qtiles;
    const int qt = p.n_qtiles - 1 - (blockIdx.x - bh * p.n_qtiles);  // heaviest query tiles first
    const int n_kv = qt + 1;                                          // tiles 0 .. diagonal

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 1);
        mbar_init(bar(B_KFULL), 1);
        mbar_init(bar(B_VFULL), 1);
        mbar_init(bar(B_KEMPTY), 1);
        mbar_init(bar(B_VEMPTY), 1);
        mbar_init(bar(B_SFULL), 1);
        mbar_init(bar(B_PFULL), 128);
        mbar_init(bar(B_OFULL), 1);
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

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer + MMA issuer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapQ) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
            auto load_k = [&](int j) {
                mbar_expect_tx(bar(B_KFULL), TILE_BYTES);
                for (int bx = 0; bx < NB; ++bx) tma_load_3d(sK + bx * kBoxBytes, &mapK, bar(B_KFULL), bx * 64, j * BN, bh);
            };
            auto load_v = [&](int j) {
                mbar_expect_tx(bar(B_VFULL), TILE_BYTES);
                for (int bx = 0; bx < NB; ++bx) tma_load_3d(sV + bx * kBoxBytes, &mapV, bar(B_VFULL), bx * 64, j * BN, bh);
            };
            // S_j = Q K_j^T.  It overwrites the columns P_{j-1} lived in: MMAs of one thread execute in
            // issue order, and P_{j-1} V_{j-1} is always issued before S_j.
            auto issue_s = [&]() {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
                    mma_bf16(tmem + COL_S, make_desc(sQ + off, 16, 1024), make_desc(sK + off, 16, 1024), IDESC_S, kk > 0 ? 1u : 0u);
                }
                mma_commit(bar(B_SFULL));
                mma_commit(bar(B_KEMPTY));
            };
            mbar_expect_tx(bar(B_QFULL), TILE_BYTES);
            for (int bx = 0; bx < NB; ++bx) tma_load_3d(sQ + bx * kBoxBytes, &mapQ, bar(B_QFULL), bx * 64, qt * BM, bh);
            load_k(0);
            load_v(0);
            bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, p.dev_status) &&
                      mbar_wait(bar(B_KFULL), 0, abort_flag, p.dev_status);
            if (ok) {
                tc_fence_after();
                issue_s();
            }
            for (int j = 0; ok && j < n_kv; ++j) {
                const bool more = j + 1 < n_kv;
                if (more) {  // K_{j+1} may land once S_j has consumed K_j
                    ok = mbar_wait(bar(B_KEMPTY), j & 1, abort_flag, p.dev_status);
                    if (!ok) break;
                    load_k(j + 1);
                }
                ok = mbar_wait(bar(B_PFULL), j & 1, abort_flag, p.dev_status) &&
                     mbar_wait(bar(B_VFULL), j & 1, abort_flag, p.dev_status);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk) {
                    // A = P from tensor memory: 16 kv columns = 8 packed 32-bit columns;
                    // B = V, MN-major: 16 kv rows = 2048 bytes; next 64 head dims one box further
                    mma_bf16_ts(tmem + COL_O, tmem + COL_S + kk * 8, make_desc(sV + kk * 2048, kBoxBytes, 1024), IDESC_O,
                                (j > 0 || kk > 0) ? 1u : 0u);
                }
                mma_commit(bar(B_VEMPTY));
                if (!more) {
                    mma_commit(bar(B_OFULL));
                    break;
                }
                // queue S_{j+1} behind P_j V_j so the tensor pipe never waits for this thread
                ok = mbar_wait(bar(B_KFULL), (j + 1) & 1, abort_flag, p.dev_status);
                if (!ok) break;
                tc_fence_after();
                issue_s();
                // V_{j+1} may land once P_j V_j has consumed V_j
                ok = mbar_wait(bar(B_VEMPTY), j & 1, abort_flag, p.dev_status);
                if (!ok) break;
                load_v(j + 1);
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: thread = query row
        const int row = threadIdx.x;                       // TMEM lane
        const int grow = qt * BM + row;                    // query block index within the sequence
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        float m_ref = kNegInf, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_kv; ++j) {
            const bool diag = (j == qt);
            ok = mbar_wait(bar(B_SFULL), j & 1, abort_flag, p.dev_status);  // S_j ready; O settled (all earlier MMAs done)
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = lane_base + COL_S;
            // On the diagonal tile the rows of warp w (32w .. 32w+31) see nothing right of column
            // 32w+31: only column chunks 0..w are loaded and exponentiated, chunk w with a per-row mask.
            const int nch = diag ? warp + 1 : BN / 32;
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
                    if (c == warp) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i > lane) sr[c * 32 + i] = __float_as_uint(kNegInf);
                    }
            }
            float mx = kNegInf;
#pragma unroll
            for (int c = 0; c < BN / 32; ++c)
                if (c < nch) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2)
                        mx = fmax3(mx, __uint_as_float(sr[c * 32 + i]), __uint_as_float(sr[c * 32 + i + 1]));
                }
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
                        tmem_ld32(lane_base + COL_O + c0, o);
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= factor;
                        tmem_st32(lane_base + COL_O + c0, o);
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
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const uint32_t* e = sr + c * 32 + i;
                        float x0, x1, x2, x3;
                        unpack2(ffma2(pack2(__uint_as_float(e[0]), __uint_as_float(e[1])), sc2, nm2), x0, x1);
                        unpack2(ffma2(pack2(__uint_as_float(e[2]), __uint_as_float(e[3])), sc2, nm2), x2, x3);
                        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
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
            mbar_arrive(bar(B_PFULL));
        }
        if (ok) ok = mbar_wait(bar(B_OFULL), 0, abort_flag, p.dev_status);
        if (ok) {
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            bf16* orow = reinterpret_cast<bf16*>(p.out) + ((size_t)bh * p.T + grow) * HD;
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
                float o[32];
                tmem_ld32(lane_base + COL_O + c0, o);
                if (grow < p.T) {
#pragma unroll
                    for (int q8 = 0; q8 < 4; ++q8) {
                        float f[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) f[i] = o[q8 * 8 + i] * inv;
                        *reinterpret_cast<uint4*>(orow + c0 + q8 * 8) = pack8(f);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---- host side: tensor maps through the driver entry point (no link-time dependency on libcuda)
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn encode_fn()
{
    static EncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(f);
    }
    return fn;
}

// [slabs][rows][hd] bf16 with `stride_rows` rows between slabs; box = 64 x 128 x 1, 128-byte swizzle,
// rows past `rows` read as zeros.
static bool make_map(CUtensorMap* m, const void* ptr, int hd, int rows, long long stride_rows, long long slabs)
{
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)hd, (cuuint64_t)rows, (cuuint64_t)slabs};
    cuuint64_t strides[2] = {(cuuint64_t)hd * 2, (cuuint64_t)stride_rows * hd * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int HD>
static cudaError_t launch_t(const PrefillArgs& a, uint32_t* dev_status, cudaStream_t stream)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(block_prefill_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             smem_bytes<HD>());
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const long long slabs = (long long)a.B * a.H;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, a.q, HD, a.T, a.T, slabs) || !make_map(&mk, a.k, HD, a.T, a.kv_seq_stride, slabs) ||
        !make_map(&mv, a.v, HD, a.T, a.kv_seq_stride, slabs))
        return cudaErrorInvalidValue;
    Params p;
    p.out = a.out;
    p.dev_status = dev_status;
    p.T = a.T;
    p.n_qtiles = (a.T + BM - 1) / BM;
    p.scale_log2 = a.scale_log2;
    const long long ctas = slabs * p.n_qtiles;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    block_prefill_tc_kernel<HD><<<(unsigned)ctas, kThreads, smem_bytes<HD>(), stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace pf

bool prefill_tc_supported(const PrefillArgs& a)
{
    auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return (a.hd == 64 || a.hd == 128) && al(a.q) && al(a.k) && al(a.v) && al(a.out) && pf::encode_fn() != nullptr;
}

cudaError_t launch_block_prefill_tc(const PrefillArgs& a, uint32_t* dev_status, cudaStream_t stream)
{
    return a.hd == 64 ? pf::launch_t<64>(a, dev_status, stream) : pf::launch_t<128>(a, dev_status, stream);
}

}  // namespace bt
