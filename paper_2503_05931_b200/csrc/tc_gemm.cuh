// Tensor-core GEMM for sm_100a: TMA-fed tcgen05.mma with the accumulator in tensor memory.
//
//   D[128 x N] (fp32, TMEM) = sum over this CTA's k-blocks of  A_tile[128 x 64] . B_tile[N x 64]^T
//
// Both operands are K-major bf16 in global memory and arrive in shared memory through
// cp.async.bulk.tensor (no multicast) with the 128-byte swizzle the MMA descriptors name.
// One CTA = one (128-row tile of A, N-row tile of B, k-split).  Warp roles: warps 0..3 issue TMA (a thread's
// copies complete one after the other, about a third of a microsecond each, so the k-blocks are shared out round
// robin over four issuing threads), warp 4 owns the TMEM allocation and issues the MMAs, warps 5..8 drain the
// accumulator (warp w reads TMEM lanes 32*(w%4) .. +31) and run the epilogue.
//
// Two uses:
//   * vocabulary projection ("weights as A"): A = output matrix [vocab, K], B = the final LayerNorm output
//     [rows, K] as a bf16 high plane and a low (residual) plane accumulated into the same D, so that
//     activations keep ~16 mantissa bits; the greedy argmax is taken in the epilogue.
//   * cross-K/V precompute ("frames as A"): A = packed encoder frames, B = [2d, d_enc] weights of a layer.
//
// Every wait on an mbarrier is bounded: on expiry the CTA raises the error word in the decode state, stops
// issuing work, waits (bounded) for its own TMA copies, frees its TMEM and returns.
#pragma once
#include <cuda.h>

#include "bounded_wait.h"
#include "common.cuh"

namespace aed {
namespace tc {

constexpr int kBlockK = 64;                    // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kTileM = 128;
constexpr int kATileBytes = kTileM * kBlockK * 2;
constexpr int kMaxStages = 8;
constexpr int kThreads = 416;                    // 8 producer warps, 1 MMA warp, 4 epilogue warps
constexpr int kProducerWarps = 8;                // (a k-block is three copies, and a thread's copies complete one after the other)
constexpr long long kWaitCycles = 2000000000ll;   // about a second at B200 clocks
constexpr int kErrTimeout = 2;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the phase did not complete in time or another role already gave up.
// (The polling loop is kept out of line: the common case is that the phase has already completed.)
__device__ __noinline__ bool mbar_wait_poll(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    return bounded_poll([&] { return mbar_try_wait(bar, parity); }, [] { return clock64(); }, kWaitCycles, abort_flag);
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_poll(bar, parity, abort_flag);
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c_inner, int c_outer, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c_inner), "r"(c_outer), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr)
{
    uint64_t desc = static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    desc |= static_cast<uint64_t>(1) << 16;            // leading byte offset (unused for swizzled K-major), 16 B
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;    // stride byte offset between 8-row groups
    desc |= static_cast<uint64_t>(1) << 46;            // descriptor version of this architecture
    desc |= static_cast<uint64_t>(2) << 61;            // 128-byte swizzle
    return desc;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__device__ __forceinline__ uint32_t instr_desc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTileM >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

enum TcEpilogue { TC_EPI_LOGITS = 1 };

struct TcParams {
    int a_rows;          // valid rows of A (output features, or frames)
    int n_tile;          // rows of B per CTA = MMA N (multiple of 16, at most 256)
    int k_blocks;        // k-blocks over the whole K
    int use_lo;          // 1: accumulate the low activation plane as well
    int rows_fixed;      // >= 0: number of valid B rows; < 0: read it from the decode state
    const __nv_bfloat16 *bias;         // over the columns of D's first dimension (vocabulary / K-V features), may be null
    // TC_EPI_LOGITS
    float *logits_out;                 // [batch, vocab] by utterance or nullptr
    unsigned long long *keys;          // [rows]
    const int32_t *active_list;
    DecState *state;
};

// grid: x = 128-row tiles of A, y = k-splits, z = N-row tiles of B.  Dynamic shared memory: stage ring + 1024.
template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_b_lo, TcParams p, int stages, int producers)
{
    // `stages` is a multiple of `producers` (1..kProducerWarps): every ring stage is refilled by one thread only, so
    // a producer is never more than one phase ahead of the barrier it waits on (a parity wait cannot tell more).
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages];
    __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
    __shared__ __align__(8) uint64_t bar_done;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    AED_TRACE_BEGIN(p.state, 16 + EPI);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = blockIdx.z * p.n_tile;
    // Only row tiles after the first can be empty; the first one skips this read so that set-up and the first
    // loads do not wait on it (the epilogue reads the row count when it needs it).
    if (blockIdx.z > 0 && row0 >= (p.rows_fixed >= 0 ? p.rows_fixed : p.state->n_active)) return;
    const int a0 = blockIdx.x * kTileM;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * blockIdx.y) / gridDim.y);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (blockIdx.y + 1)) / gridDim.y);
    const int n_kb = kb_end - kb_begin;
    if (n_kb <= 0) return;

    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const int b_bytes = p.n_tile * kBlockK * 2;
    const int planes = p.use_lo ? 2 : 1;
    const int stage_bytes = kATileBytes + planes * b_bytes;
    uint32_t tmem_cols = 32;
    while (tmem_cols < static_cast<uint32_t>(p.n_tile)) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_done, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&tmem_slot, tmem_cols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (threadIdx.x == 0) AED_TRACE_MARK(p.state, 32);      // set-up done
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp < kProducerWarps) {
        if (lane == 0 && warp < producers) {
            prefetch_tensormap(&map_a);
            prefetch_tensormap(&map_b);
            if (p.use_lo) prefetch_tensormap(&map_b_lo);
            int issued = 0;
            bool waited = false;
            for (int i = warp; i < n_kb; i += producers) {
                const int s = i % stages;
                if (i >= stages && !mbar_wait(&bar_empty[s], ((i / stages) - 1) & 1, &abort_flag)) break;
                uint8_t *st = tiles + static_cast<size_t>(s) * stage_bytes;
                mbar_expect_tx(&bar_full[s], stage_bytes);
                const int kc = (kb_begin + i) * kBlockK;
                tma_load_2d(st, &map_a, kc, a0, &bar_full[s]);
                // A is static (a weight matrix): its first tile is requested while the previous kernel still runs;
                // B is that kernel's output
                if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
                tma_load_2d(st + kATileBytes, &map_b, kc, row0, &bar_full[s]);
                if (p.use_lo) tma_load_2d(st + kATileBytes + b_bytes, &map_b_lo, kc, row0, &bar_full[s]);
                issued = i + 1;
            }
            if (abort_flag && issued > 0) {
                // give this thread's last copies a bounded chance to land before the CTA's memory goes away
                const int i = issued - 1;
                const long long start = clock64();
                while (!mbar_try_wait(&bar_full[i % stages], (i / stages) & 1) && clock64() - start < kWaitCycles / 8) {}
            }
        }
    } else if (warp == kProducerWarps) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(p.n_tile);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % stages;
                ok = mbar_wait(&bar_full[s], (i / stages) & 1, &abort_flag);
                if (!ok) break;
                if (i == 0) AED_TRACE_MARK(p.state, 33);    // first operands landed
                tc_fence_after_sync();
                const uint32_t sa = smem_u32(tiles + static_cast<size_t>(s) * stage_bytes);
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + kATileBytes);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k)
                    mma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                if (p.use_lo) {
                    const uint64_t dl = smem_desc_sw128(sa + kATileBytes + b_bytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(tmem_base, da + 2 * k, dl + 2 * k, idesc, 1u);
                }
                mma_commit(&bar_empty[s]);      // the stage may be refilled once these MMAs have read it
            }
            if (ok) mma_commit(&bar_done);      // accumulator complete
        }
    } else {
        // epilogue warps
        const int quarter = warp & 3;
        const int n_rows = p.rows_fixed >= 0 ? p.rows_fixed : p.state->n_active;
        const bool ok = mbar_wait(&bar_done, 0, &abort_flag);
        tc_fence_after_sync();
        if (threadIdx.x == (kProducerWarps + 1) * 32) AED_TRACE_MARK(p.state, 34);  // accumulator complete
        if (ok) {
            const int a_idx = a0 + quarter * 32 + lane;          // row of A this thread owns
            const bool a_ok = a_idx < p.a_rows;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            if (EPI == TC_EPI_LOGITS) {
                const float bias = (p.bias && a_ok) ? to_f32(p.bias[a_idx]) : 0.f;
                for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int r = row0 + c0 + j;                 // uniform over the warp
                        if (r >= n_rows) continue;
                        const float z = v[j] + bias;
                        if (p.logits_out && a_ok) p.logits_out[static_cast<size_t>(p.active_list[r]) * p.a_rows + a_idx] = z;
                        // warp maximum of the order-preserving key, then the lowest lane that attains it
                        const uint32_t k32 = a_ok ? float_order_key(z) : 0u;
                        const uint32_t kmax = __reduce_max_sync(0xffffffffu, k32);
                        const uint32_t winners = __ballot_sync(0xffffffffu, k32 == kmax);
                        const uint32_t best = a0 + quarter * 32 + (__ffs(winners) - 1);
                        const unsigned long long key =
                            kmax ? ((static_cast<unsigned long long>(kmax) << 32) | (0xFFFFFFFFu - best)) : 0ull;
                        if (lane == 0 && key != 0ull) atomicMax(p.keys + r, key);
                    }
                }
            }
        }
    }
    if (threadIdx.x == (kProducerWarps + 1) * 32) AED_TRACE_MARK(p.state, 35);      // epilogue issued
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kProducerWarps) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(&p.state->error, kErrTimeout);
}

}  // namespace tc
}  // namespace aed
