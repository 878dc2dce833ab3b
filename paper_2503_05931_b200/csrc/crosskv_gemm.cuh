// Cross-attention K/V of every layer in one persistent tensor-core GEMM (sm_100a).
//
//   store[l][k|v][head][frame][64] = bf16( enc[frame, :] . w_kv_c[l][feature, :] + b_kv_c[l][feature] )
// (or rounded to the 8-bit format E4M3 instead of bf16 when the handle stores the cross-attention K/V in 8 bits)
//
// over the packed encoder frames (no padding rows).  One block per SM walks a list of output tiles
// (128 frames x 256 features, K = d_enc in 64-wide k-blocks).  Tile order: groups of gridDim.x frame tiles outermost;
// inside a group the tiles are numbered (layer, feature tile) major, frame tile minor, and block b takes the numbers
// b, b + gridDim.x, ...  With a full group block b therefore keeps frame tile group * gridDim.x + b for every layer
// and feature tile: the frame tiles of a group stay in L2 while all layers' weights stream past them, and the
// weights are re-read once per group only.  With fewer frame tiles than blocks the same numbering spreads the
// (layer, feature tile) pairs over the idle blocks.
//
// Warp roles (12 warps): 0..3 producers, 4 issues the MMAs, 5..7 idle, 8..11 epilogue.
//   * A thread's TMA copies complete one after the other (about a third of a microsecond each on this part,
//     whatever their size), so one issuing thread cannot feed the tensor cores: four producer threads share the
//     k-blocks round robin, each loading both operands of its k-blocks into a ring of 48 KB stages.
//   * The accumulator (128 lanes x 256 fp32 columns) is double-buffered in tensor memory: while the epilogue
//     warps drain tile i (bias, bf16 pack, 16-byte stores straight into the per-head K/V rows), the MMA warp
//     already accumulates tile i + 1.
// Every wait is bounded; on expiry the block raises the sticky error word, lets its copies land, frees its tensor
// memory and returns.
#pragma once
#include "tc_gemm.cuh"

namespace aed {
namespace ckv {

using namespace tc;

constexpr int kTileN = 256;                       // features per tile = MMA N
constexpr int kStageBytes = kATileBytes + kTileN * kBlockK * 2;      // 16 KB frames + 32 KB weights
constexpr int kStages = 4;
constexpr int kProducers = 4;
constexpr int kCkvThreads = 384;
constexpr int kMaxLayers = 64;

// The frames of a launch: up to kMaxSegs runs of consecutive rows of the encoder tensor, each with a store row of its
// own (a packed batch is one run; utterances admitted into slots are one run each).  Frame tiles never straddle runs.
constexpr int kMaxSegs = 16;
struct CkvSegs {
    int n;
    int tile0[kMaxSegs + 1];          // first frame tile of every run, and the total
    int src0[kMaxSegs];               // row of the run's first frame in the encoder tensor
    int frames[kMaxSegs];
    int dst0[kMaxSegs];               // store row of the run's first frame
};

struct CkvParams {
    CkvSegs segs;
    int frame_capacity;
    int d_model, n_heads, d_enc;
    int n_layers;
    void *store;                      // layer 0; layers are layer_elems elements apart; bf16, or E4M3 bytes (template argument)
    size_t layer_elems;
    const __nv_bfloat16 *const *bias; // [n_layers] device pointers (entries may be null), or null
    DecState *state;
};

// The tiles of one block, in order.  Every warp role walks the same sequence.
struct TileWalk {
    int m_tiles, per_group, G, b;
    int group, gsize;
    long long id, total;
    __device__ TileWalk(int m_tiles_, int per_group_, int G_, int b_) : m_tiles(m_tiles_), per_group(per_group_), G(G_), b(b_)
    {
        group = 0;
        gsize = min(G, m_tiles);
        total = static_cast<long long>(per_group) * gsize;
        id = b;
        settle();
    }
    __device__ void settle()
    {
        while (gsize > 0 && id >= total) {          // next group
            ++group;
            gsize = min(G, m_tiles - group * G);
            if (gsize <= 0) { gsize = 0; break; }
            total = static_cast<long long>(per_group) * gsize;
            id = b;
        }
    }
    __device__ bool valid() const { return gsize > 0; }
    __device__ int lnt() const { return static_cast<int>(id / gsize); }                       // layer * n_tiles + feature tile
    __device__ int m_tile() const { return group * G + static_cast<int>(id % gsize); }
    __device__ void next() { id += G; settle(); }
};

// grid: persistent blocks.  map_w: one tensor map per layer over w_kv_c [2d, d_enc], boxes of 256 rows x 64.
template <bool kE4M3>
__global__ void __launch_bounds__(kCkvThreads, 1)
crosskv_gemm_kernel(const __grid_constant__ CUtensorMap map_enc, const CUtensorMap *__restrict__ map_w, const __grid_constant__ CkvParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_full[kStages];
    __shared__ __align__(8) uint64_t bar_empty[kStages];
    __shared__ __align__(8) uint64_t bar_acc_full[2];     // accumulator buffer complete (MMA -> epilogue)
    __shared__ __align__(8) uint64_t bar_acc_free[2];     // accumulator buffer drained (epilogue -> MMA)
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const int k_blocks = p.d_enc / kBlockK;
    const int m_tiles = p.segs.tile0[p.segs.n];
    // run and tile inside the run of a frame tile
    auto locate = [&](int m_tile, int &seg, int &j) {
        seg = 0;
        while (seg + 1 < p.segs.n && m_tile >= p.segs.tile0[seg + 1]) ++seg;
        j = m_tile - p.segs.tile0[seg];
    };
    const int n_tiles = (2 * p.d_model + kTileN - 1) / kTileN;
    const int per_group = p.n_layers * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bar_acc_full[b], 1); mbar_init(&bar_acc_free[b], 4); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(&tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    if (warp < kProducers) {
        if (lane == 0) {
            prefetch_tensormap(&map_enc);
            long long it = 0;                           // k-block counter over all of this block's tiles
            bool ok = true;
            long long issued_last = -1;
            for (TileWalk w(m_tiles, per_group, gridDim.x, blockIdx.x); w.valid() && ok; w.next()) {
                const int layer = w.lnt() / n_tiles, nt = w.lnt() % n_tiles;
                int seg, j;
                locate(w.m_tile(), seg, j);
                const int m0 = p.segs.src0[seg] + j * kTileM;          // rows past the run's end are loaded and never stored
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    if (static_cast<int>(it % kProducers) != warp) continue;
                    const int s = static_cast<int>(it % kStages);
                    if (it >= kStages && !mbar_wait(&bar_empty[s], static_cast<uint32_t>((it / kStages) - 1) & 1, &abort_flag)) { ok = false; break; }
                    uint8_t *st = tiles + static_cast<size_t>(s) * kStageBytes;
                    mbar_expect_tx(&bar_full[s], kStageBytes);
                    tma_load_2d(st, &map_enc, kb * kBlockK, m0, &bar_full[s]);
                    tma_load_2d(st + kATileBytes, map_w + layer, kb * kBlockK, nt * kTileN, &bar_full[s]);
                    issued_last = it;
                }
            }
            if (!ok && issued_last >= 0) {
                // gave up: give this thread's last copy a bounded chance to land before the block's memory goes away
                const long long start = clock64();
                while (!mbar_try_wait(&bar_full[issued_last % kStages], static_cast<uint32_t>(issued_last / kStages) & 1) &&
                       clock64() - start < kWaitCycles / 8) {}
            }
        }
    } else if (warp == 4) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(kTileN);
            long long it = 0;
            bool ok = true;
            long long t = 0;
            for (TileWalk w(m_tiles, per_group, gridDim.x, blockIdx.x); w.valid() && ok; w.next(), ++t) {
                const int buf = static_cast<int>(t & 1);
                // the epilogue must have drained this buffer (its previous use was tile t - 2)
                if (t >= 2) ok = mbar_wait(&bar_acc_free[buf], static_cast<uint32_t>((t >> 1) - 1) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t acc = tmem_base + static_cast<uint32_t>(buf * kTileN);
                for (int kb = 0; kb < k_blocks && ok; ++kb, ++it) {
                    const int s = static_cast<int>(it % kStages);
                    ok = mbar_wait(&bar_full[s], static_cast<uint32_t>(it / kStages) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(tiles + static_cast<size_t>(s) * kStageBytes);
                    const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(acc, da + 2 * k, db + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    mma_commit(&bar_empty[s]);
                }
                if (ok) mma_commit(&bar_acc_full[buf]);
            }
        }
    } else if (warp >= 8) {
        // epilogue: warp w reads TMEM lanes 32 * (w & 3) .. + 31; this thread owns one frame of the tile
        const int quarter = warp & 3;
        bool ok = true;
        long long t = 0;
        for (TileWalk w(m_tiles, per_group, gridDim.x, blockIdx.x); w.valid() && ok; w.next(), ++t) {
            const int layer = w.lnt() / n_tiles, nt = w.lnt() % n_tiles;
            int seg, j;
            locate(w.m_tile(), seg, j);
            const int frame_in_run = j * kTileM + quarter * 32 + lane;
            const bool frame_ok = frame_in_run < p.segs.frames[seg];
            const int frame = p.segs.dst0[seg] + frame_in_run;
            const int buf = static_cast<int>(t & 1);
            ok = mbar_wait(&bar_acc_full[buf], static_cast<uint32_t>(t >> 1) & 1, &abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + static_cast<uint32_t>(buf * kTileN) + (static_cast<uint32_t>(quarter * 32) << 16);
            const size_t layer_off = static_cast<size_t>(layer) * p.layer_elems;
            const __nv_bfloat16 *bias = p.bias ? p.bias[layer] : nullptr;
            for (int c0 = 0; c0 < kTileN; c0 += 16) {
                float v[16];
                tmem_ld16(taddr + c0, v);
                const int o = nt * kTileN + c0;                  // 16 consecutive features inside one head
                if (!frame_ok || o >= 2 * p.d_model) continue;
                const int kv = o / p.d_model, cc = o % p.d_model, h = cc / kHeadDim, e = cc % kHeadDim;
                if (bias) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += to_f32(bias[o + j]);
                }
                const size_t elem = layer_off + ((static_cast<size_t>(kv) * p.n_heads + h) * p.frame_capacity + frame) * kHeadDim + e;
                uint32_t packed[8];
                if (kE4M3) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        packed[j] = static_cast<uint32_t>(pack_e4m3x2(v[4 * j], v[4 * j + 1])) |
                                    (static_cast<uint32_t>(pack_e4m3x2(v[4 * j + 2], v[4 * j + 3])) << 16);
                    *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(p.store) + elem) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        __nv_bfloat162 pair = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                        packed[j] = *reinterpret_cast<uint32_t *>(&pair);
                    }
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.store) + elem;
                    reinterpret_cast<uint4 *>(dst)[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    reinterpret_cast<uint4 *>(dst)[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
                }
            }
            // this warp is done with the buffer
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_acc_free[buf])) : "memory");
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(&p.state->error, kErrTimeout);
}

}  // namespace ckv
}  // namespace aed
