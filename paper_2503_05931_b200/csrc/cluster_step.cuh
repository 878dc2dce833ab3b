// Head-parallel decode step for small batches (at most 64 rows): three cluster kernels per layer.
//
// A decoder layer has three places where every output needs the whole residual row x: before the self-attention
// projections (LN1), before the cross-attention query projection (LN2) and before the feed-forward network (LN3).
// Everything between two such places can be split over attention heads (or over slices of the FFN hidden layer)
// without any exchange between the parts, so a layer is run as three "blocks":
//
//   K_SELF   x_out = x_in + Wo  . selfattn (LN1(x_in))      cluster = (head, rows of one parity)
//   K_CROSS  x_out = x_in + Woc . crossattn(LN2(x_in))      cluster = (head, rows of one parity)
//   K_FFN    x_out = x_in + W2 . relu(W1 . LN3(x_in) + b1) + b2      cluster = 128 hidden features, all rows
//
// Each block is one launch of 32 clusters of 4 CTAs (a B200 holds 36 such clusters at once, but only 15 clusters
// of 8).  Inside a cluster the 4 CTAs split the contraction dimension of the first projection (K = d_model, d/4
// columns each) and the output features of the second one (d/4 each); partial results travel through distributed
// shared memory:
//
//   1. every CTA loads its d/4 columns of x_in for the cluster's rows, folds the LayerNorm scale in (gamma*x, bf16
//      high and low planes) and computes the (mean, M2) of its slice of every row;
//   2. tcgen05.mma: partial[feature, row] over the CTA's K slice (weights are the A operand, fetched by TMA before
//      the dependency wait because they are static);
//   3. the partials are scattered to the CTA that owns the row (attention blocks: local row l belongs to CTA l mod 4)
//      or the hidden feature (FFN: 32 features per CTA), together with the slice statistics; an mbarrier with
//      cluster-scope release/acquire marks the end of the exchange;
//   4. the owner sums the 4 partials, finishes the LayerNorm (rstd*(raw - mean*c1) + c2, see step_gemm.cuh) and
//      runs attention for its rows over the ragged cache (or applies ReLU), then writes the result as bf16 planes
//      straight into the B-operand tile of all 4 CTAs;
//   5. tcgen05.mma of the second projection over the head's 64 (or the chunk's 128) input features, d/4 output
//      features per CTA, and 16-byte red.global.add of the partial into x_out, which an earlier block cleared.
//
// x rotates through three buffers (read, accumulate, clear) so that a fast cluster can never add into rows that a
// slow cluster of the same launch still reads.  Only the sum over heads / hidden chunks goes through global
// memory: three exchanges per layer instead of eight.
//
// Attention inside a CTA: the 16-position chunks of its rows form one list that is dealt to the 8 worker warps in
// equal contiguous runs; each warp streams its chunks through a ring in shared memory filled by bulk async copies
// (the first stages before the dependency wait, since cached keys and values are static during a step).
//
// Every wait is bounded; a CTA that gives up still performs all its cluster arrivals, so that its peers do not
// wait for it, and raises the error word of the decode state.
#pragma once
#include "step_gemm.cuh"
#include "step_kernels.cuh"

namespace aed {
namespace cl {

using namespace tc;

constexpr int kCS = 4;               // CTAs per cluster
constexpr int kClusters = 32;
constexpr int kClThreads = 384;      // warp 0 TMA, warp 1 MMA, warps 2..9 workers, warps 10..11 side jobs
constexpr int kSlot = 16384;         // one weight tile: 128 rows x 64 k, bf16
constexpr int kMaxTiles = 10;
constexpr int kMaxRing = 4;
constexpr int kMaxRows = 64;
constexpr int kMaxSlots = 8;         // rows of one CTA in an attention block
constexpr int kFfnSlots = 7;         // weight slots of the FFN block
constexpr int kTmemCols = 256;

enum Kind { K_SELF = 0, K_CROSS = 1, K_FFN = 2 };

struct ClusterParams {
    int d, n_heads, d_ffn, n_tile;
    const float *x_in;
    float *x_out, *x_zero;
    const __nv_bfloat16 *gamma;        // LayerNorm scale of this block [d]
    const float *c1, *c2;              // fold constants of the first projection, indexed by its output feature
    const __nv_bfloat16 *bias2;        // bias of the second projection [d], may be null
    __nv_bfloat16 *cache;              // K_SELF: self cache of this layer; K_CROSS: cross store of this layer
    int seq_capacity;
    const int4 *row_info;
    float scale, eps;
    DecState *state;
    // static data the next block streams: pulled into L2 before the dependency wait
    const void *pf_ptr[2];
    size_t pf_bytes[2];
    const __nv_bfloat16 *pf_cache;     // K/V rows of the next attention block (null: none)
    int pf_capacity, pf_cross;
};

struct ClSmem {
    int recv_off, r2_off, ap_off, stats_off, tab_off, ring_off, ring_stages, total;
};

constexpr int kRingStage = 4096;                // 16 positions: keys 2 KB | values 2 KB
constexpr int kPartStride = 68;                 // floats per attention partial: max, sum, pad, pad, 64 accumulators
constexpr int kDynSmemCap = 232448 - 3072;      // what a CTA may take, less the static part of the kernel

// MMA N of a block: the attention blocks see every second row of the step
__host__ __device__ inline int cl_mma_n(int kind, int n_tile) { return kind == K_FFN ? n_tile : (n_tile / 2 < 16 ? 16 : n_tile / 2); }

// Byte offset of weight tile t in the weight area (kbs = k-blocks of the CTA's K slice, mt2 = 128-row tiles of its
// output features).  Tiles of 64 rows take 8 KB; the MMA reads 128 rows from the tile base whatever follows it
// (rows 64..127 only feed accumulator lanes nobody reads).
//   K_SELF : per k-block  query|key rows 16 KB, value rows 8 KB; the output-projection tiles later reuse the
//            query|key areas of the first k-blocks
//   K_CROSS: query tiles 8 KB each, then the output-projection tiles
//   K_FFN  : 7 slots of 16 KB, tile t in slot t mod 7
__host__ __device__ inline int cl_tile_off(int kind, int t, int kbs)
{
    if (kind == K_SELF) return t < 2 * kbs ? (t >> 1) * 24576 + (t & 1) * 16384 : (t - 2 * kbs) * 24576;
    if (kind == K_CROSS) return t < kbs ? t * 8192 : kbs * 8192 + (t - kbs) * kSlot;
    return (t % kFfnSlots) * kSlot;
}

// Dynamic shared memory of one block kind:
// weight tiles | receive buffer (later: attention partials) | operand planes | attention planes | statistics |
// attention tables | K/V ring (8 warps x stages x 4 KB)
__host__ __device__ inline ClSmem cl_layout(int kind, int n_tile, int kbs)
{
    ClSmem s;
    const int mt2 = kbs / 2, nm = cl_mma_n(kind, n_tile);
    const int tiles_ffn = kbs + 2 * mt2;
    const int w_bytes = kind == K_SELF ? kbs * 24576 : kind == K_CROSS ? kbs * 8192 + mt2 * kSlot
                                                                        : (tiles_ffn < kFfnSlots ? tiles_ffn : kFfnSlots) * kSlot;
    int recv = kind == K_SELF ? n_tile * 384 : kind == K_CROSS ? n_tile * 272 : n_tile * 512;
    recv = (recv + 1023) / 1024 * 1024;
    const int r2 = kbs * 2 * nm * 128;
    const int ap = kind == K_FFN ? 0 : 2 * nm * 128;
    s.recv_off = w_bytes;
    s.r2_off = s.recv_off + recv;
    s.ap_off = s.r2_off + r2;
    s.stats_off = s.ap_off + ap;
    s.tab_off = s.stats_off + kCS * kMaxRows * 8;
    s.ring_off = s.tab_off + (kind == K_FFN ? 0 : 5120);
    s.ring_stages = 0;
    if (kind != K_FFN) {
        int st = (kDynSmemCap - s.ring_off - 1024) / (8 * kRingStage);
        s.ring_stages = st < 1 ? 1 : st > kMaxRing ? kMaxRing : st;
    }
    s.total = s.ring_off + s.ring_stages * 8 * kRingStage;
    return s;
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_index()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in the CTA with the given rank of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x2(uint32_t addr, float a, float b)
{
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void st_cluster_b128(uint32_t addr, uint4 v)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void arrive_remote(uint32_t remote_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long start = clock64();
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - start > kWaitCycles) { *abort_flag = 1; return false; }
    }
}
// all threads of all CTAs of the cluster
__device__ __forceinline__ void cluster_sync_all()
{
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
// contiguous global -> shared copy by the async engine; completes on an mbarrier of this CTA
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// (mean, rstd) of a row from the (mean, M2) of its equally long slices, one per CTA of the cluster
__device__ __forceinline__ float2 merge_stats(const float2 *slices, int stride, int ks, int d, float eps)
{
    float2 s[kCS];
    float mean = 0.f;
#pragma unroll
    for (int i = 0; i < kCS; ++i) { s[i] = slices[i * stride]; mean += s[i].x; }
    mean *= (1.f / kCS);
    float m2 = 0.f;
#pragma unroll
    for (int i = 0; i < kCS; ++i) { const float dm = s[i].x - mean; m2 += s[i].y + ks * dm * dm; }
    return make_float2(mean, rsqrtf(m2 / d + eps));
}

// 8 floats through L2 only (rows that other CTAs of a persistent launch wrote earlier in the same launch)
__device__ __forceinline__ void load8_cg(const float *p, float (&v)[8])
{
    const float4 a = __ldcg(reinterpret_cast<const float4 *>(p));
    const float4 b = __ldcg(reinterpret_cast<const float4 *>(p + 4));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// mbarriers of one block kind; each completes one phase per block of that kind (parity = number of earlier uses & 1)
struct BlockBars {
    uint64_t w[kMaxTiles];     // one per weight tile
    uint64_t b, d1, d2;        // operand planes written; first / second projection complete
    uint64_t c0, c1;           // first / second exchange of the cluster
};

// Static shared state of a CTA, common to all blocks it runs.
struct CtaShared {
    BlockBars bars[3];
    uint64_t ring_bar[8][kMaxRing];                 // K/V ring of each worker warp
    uint32_t tmem_slot;
    int abort_flag;
    float c1[192], c2[192];                         // fold constants of the features this CTA finishes
    const __nv_bfloat16 *kptr[kMaxSlots], *vptr[kMaxSlots];      // per row slot of this CTA
    int len[kMaxSlots], lenst[kMaxSlots], cum[kMaxSlots + 1];
};

__device__ __forceinline__ void init_cta_shared(CtaShared &sh)
{
    for (int k = 0; k < 3; ++k) {
        BlockBars &bars = sh.bars[k];
        for (int i = 0; i < kMaxTiles; ++i) mbar_init(&bars.w[i], 1);
        mbar_init(&bars.b, 8);
        mbar_init(&bars.d1, 1);
        mbar_init(&bars.d2, 1);
        mbar_init(&bars.c0, kCS * 8);               // 8 worker warps of each CTA of the cluster
        mbar_init(&bars.c1, kCS * 8);
    }
    for (int i = 0; i < 8 * kMaxRing; ++i) mbar_init(&sh.ring_bar[0][0] + i, 1);
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// One block of a layer on this CTA.
//   par        parity of this kind's single-use barriers (how many blocks of the kind this CTA ran before, & 1)
//   ring_phase parities of the K/V ring barriers, carried from block to block
//   sync_word  PERSIST: grid-wide arrival counter; the block may read x_in once it has reached sync_target
template <int KIND, bool PERSIST>
__device__ __forceinline__ void run_block(const ClusterParams &p, const CUtensorMap *map_w1, const CUtensorMap *map_w2,
                                          int n_tile, uint32_t par, CtaShared &sh, uint8_t *smem_dyn, uint32_t tmem_base,
                                          uint32_t &ring_phase, int *sync_word, int sync_target)
{
    BlockBars &bars = sh.bars[KIND];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = static_cast<int>(cluster_ctarank());
    const int c = static_cast<int>(cluster_index());
    const int d = p.d, ks = d / kCS, kbs = ks / kBlockK, of = ks, mt2 = of / kTileM;
    const int N = n_tile;
    // attention blocks: cluster = (head, row parity); local row l is row 2 l + parity of the step
    const int head = c >> 1, parity = c & 1;
    const int Nm = cl_mma_n(KIND, N);                // MMA N = rows of the operand tiles
    const int n_work = KIND == K_FFN ? p.d_ffn / 128 : p.n_heads;      // heads / hidden chunks that exist
    const bool has_work = KIND == K_FFN ? c < n_work : head < n_work;
    const ClSmem lay = cl_layout(KIND, N, kbs);
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *w_tiles = base;
    float *recv = reinterpret_cast<float *>(base + lay.recv_off);
    uint8_t *r2 = base + lay.r2_off;                 // x planes; K_FFN: later the hidden planes
    uint8_t *ap = base + lay.ap_off;                 // attention output planes
    float2 *stats_recv = reinterpret_cast<float2 *>(base + lay.stats_off);
    float *sm_q = reinterpret_cast<float *>(base + lay.tab_off);                                  // [8][64] scaled queries
    __nv_bfloat16 *sm_knew = reinterpret_cast<__nv_bfloat16 *>(base + lay.tab_off + 2048);         // [8][64] new keys
    __nv_bfloat16 *sm_vnew = sm_knew + kMaxSlots * kHeadDim;                                       // [8][64] new values
    uint8_t *ring = base + lay.ring_off;
    float *part = recv;                              // attention partials reuse the receive buffer
    const int RS = lay.ring_stages;
    const int pb = Nm * 128;                         // bytes of one plane of one k-block
    const int n_tiles1 = KIND == K_SELF ? 2 * kbs : kbs;
    const int n_tiles2 = KIND == K_FFN ? 2 * mt2 : mt2;
    const int n_tiles = n_tiles1 + n_tiles2;


    // Everything before this call touches only data that no block of the step writes.
    auto dep_wait = [&]() {
        if (!PERSIST) {
            sg::pdl_wait();
        } else {
            if (sync_target > 0 && threadIdx.x == 64) {                 // one poller per CTA
                const long long start = clock64();
                while (true) {
                    int seen;
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(sync_word) : "memory");
                    if (seen >= sync_target || sh.abort_flag) break;
                    if (clock64() - start > kWaitCycles) { sh.abort_flag = 1; break; }
                }
            }
            asm volatile("bar.sync 2, 320;" ::: "memory");               // workers and side-job warps
        }
    };

    if (warp == 0) {
        // ---- weight tiles by TMA: static data, requested before the dependency wait ---------------------------
        if (lane == 0 && has_work) {
            prefetch_tensormap(map_w1);
            prefetch_tensormap(map_w2);
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                // tiles that reuse the area of a tile of the first projection wait for its MMAs
                if ((KIND == K_SELF && t >= n_tiles1) || (KIND == K_FFN && t >= kFfnSlots)) {
                    ok = mbar_wait(&bars.d1, par, &sh.abort_flag);
                    if (!ok) break;
                }
                uint8_t *slot = w_tiles + cl_tile_off(KIND, t, kbs);
                if (t < n_tiles1) {
                    const int kb = KIND == K_SELF ? t >> 1 : t;
                    const int kc = j * ks + kb * kBlockK;
                    if (KIND == K_SELF) {
                        if ((t & 1) == 0) {          // query rows | key rows of the head
                            mbar_expect_tx(&bars.w[t], 2 * 8192);
                            tma_load_2d(slot, map_w1, kc, head * kHeadDim, &bars.w[t]);
                            tma_load_2d(slot + 8192, map_w1, kc, d + head * kHeadDim, &bars.w[t]);
                        } else {                     // value rows
                            mbar_expect_tx(&bars.w[t], 8192);
                            tma_load_2d(slot, map_w1, kc, 2 * d + head * kHeadDim, &bars.w[t]);
                        }
                    } else if (KIND == K_CROSS) {
                        mbar_expect_tx(&bars.w[t], 8192);
                        tma_load_2d(slot, map_w1, kc, head * kHeadDim, &bars.w[t]);
                    } else {                         // the 128 hidden features of chunk c
                        mbar_expect_tx(&bars.w[t], 2 * 8192);
                        tma_load_2d(slot, map_w1, kc, c * 128, &bars.w[t]);
                        tma_load_2d(slot + 8192, map_w1, kc, c * 128 + 64, &bars.w[t]);
                    }
                } else {                             // second projection: 128 of this CTA's d/4 output features
                    const int u = t - n_tiles1;
                    const int m = KIND == K_FFN ? u >> 1 : u;
                    const int kc = KIND == K_FFN ? c * 128 + (u & 1) * kBlockK : head * kHeadDim;
                    mbar_expect_tx(&bars.w[t], 2 * 8192);
                    tma_load_2d(slot, map_w2, kc, j * of + m * kTileM, &bars.w[t]);
                    tma_load_2d(slot + 8192, map_w2, kc, j * of + m * kTileM + 64, &bars.w[t]);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue --------------------------------------------------------------------------------------------
        if (lane == 0 && has_work) {
            const uint32_t idesc = instr_desc_bf16(Nm);
            bool ok = mbar_wait(&bars.b, par, &sh.abort_flag);
            for (int t = 0; t < n_tiles1 && ok; ++t) {
                ok = mbar_wait(&bars.w[t], par, &sh.abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const int kb = KIND == K_SELF ? t >> 1 : t;
                const int acc = KIND == K_SELF ? (t & 1) : 0;
                const uint32_t sa = smem_u32(w_tiles + cl_tile_off(KIND, t, kbs));
                const uint32_t sb = smem_u32(r2 + static_cast<size_t>(kb) * 2 * pb);
                const uint64_t da = smem_desc_sw128(sa), dh = smem_desc_sw128(sb), dl = smem_desc_sw128(sb + pb);
                const uint32_t td = tmem_base + acc * Nm;
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dh + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dl + 2 * k, idesc, 1u);
            }
            if (ok) mma_commit(&bars.d1);
            // second projection: its B operand is complete when the second exchange of the cluster is
            ok = ok && mbar_wait_cluster(&bars.c1, par, &sh.abort_flag);
            if (ok) {
                fence_async_proxy();
                tc_fence_after_sync();
                for (int u = 0; u < n_tiles2 && ok; ++u) {
                    const int t = n_tiles1 + u;
                    ok = mbar_wait(&bars.w[t], par, &sh.abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int m = KIND == K_FFN ? u >> 1 : u, q = KIND == K_FFN ? (u & 1) : 0;
                    const uint32_t sa = smem_u32(w_tiles + cl_tile_off(KIND, t, kbs));
                    const uint32_t sb = smem_u32(KIND == K_FFN ? r2 + static_cast<size_t>(q) * 2 * pb : ap);
                    const uint64_t da = smem_desc_sw128(sa), dh = smem_desc_sw128(sb), dl = smem_desc_sw128(sb + pb);
                    const uint32_t td = tmem_base + (2 + m) * Nm;
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dh + 2 * k, idesc, (q > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dl + 2 * k, idesc, 1u);
                }
                if (ok) mma_commit(&bars.d2);
            }
        }
    } else if (warp >= 10) {
        // ---- side jobs -----------------------------------------------------------------------------------------------
        const int st = threadIdx.x - 320;                 // 0..63
        const int cta = blockIdx.x, n_cta = gridDim.x;
        for (int i = 0; i < 2; ++i) {
            if (!p.pf_ptr[i]) continue;
            const size_t pieces = p.pf_bytes[i] / 4096;
            const char *src = static_cast<const char *>(p.pf_ptr[i]);
            for (size_t k = static_cast<size_t>(cta) * 64 + st; k < pieces; k += static_cast<size_t>(n_cta) * 64)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + k * 4096), "r"(4096) : "memory");
        }
        if (p.pf_cache && head < p.n_heads) {
            // keys and values that the (head, parity) rows of this CTA read in the next attention block:
            // thread = (row slot, k|v)
            const int slot = st >> 1, kv = st & 1;
            if (slot < N / 2 / kCS) {
                const int4 ri = p.row_info[2 * (j + kCS * slot) + parity];
                if (ri.x >= 0) {
                    const __nv_bfloat16 *src;
                    int len;
                    if (p.pf_cross) {
                        src = p.pf_cache + ((size_t)(kv * p.n_heads + head) * p.pf_capacity + ri.w) * kHeadDim;
                        len = ri.z;
                    } else {
                        src = p.pf_cache + (((size_t)ri.x * 2 + kv) * p.n_heads + head) * (size_t)p.pf_capacity * kHeadDim;
                        len = ri.y;
                    }
                    for (int off = 0; off < len; off += 32) {
                        const int rows = min(32, len - off);
                        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + (size_t)off * kHeadDim), "r"(rows * 128) : "memory");
                    }
                }
            }
        }
        dep_wait();
        if (p.x_zero) {
            const int n_rows = p.state->n_active;
            const size_t total4 = static_cast<size_t>(n_rows) * d / 4;
            float4 *z = reinterpret_cast<float4 *>(p.x_zero);
            for (size_t idx = static_cast<size_t>(cta) * 64 + st; idx < total4; idx += static_cast<size_t>(n_cta) * 64)
                z[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    } else {
        // ---- workers: 8 warps ---------------------------------------------------------------------------------
        const int ww = warp - 2, pt = threadIdx.x - 64, quarter = warp & 3;
        // timeline of the first worker thread of block 0 and of block 72
        AED_TRACE_RESERVE(tcur, p.state, (pt == 0 && (blockIdx.x == 0 || blockIdx.x == 72)) ? 96u : 0u);
        AED_TRACE_PUT(p.state, tcur, (blockIdx.x == 0 ? 24 : 124) + KIND);
        const uint32_t recv_s = smem_u32(recv), stats_s = smem_u32(stats_recv);
        const uint32_t cbar0_s = smem_u32(&bars.c0), cbar1_s = smem_u32(&bars.c1);
        const uint32_t ap_s = smem_u32(ap), r2_s = smem_u32(r2);
        // x slice geometry: thread = (local row within pass, 8-column chunk cc)
        const int cpr = ks >> 3, rows_per_pass = 256 / cpr;          // 16 or 32 chunks per row
        const int cc = pt % cpr, r_in_pass = pt / cpr;
        const int n_loc_cap = KIND == K_FFN ? N : N / 2;            // local rows of the cluster (capacity)
        const int SL = N / 2 / kCS;                        // row slots per CTA in the attention blocks: local row = j + 4 slot
        const int dg = lane & 7, pg = lane >> 3;
        float gam[8];
        // Attention work of this CTA: the 16-position chunks of all its rows, numbered row after row and dealt out
        // to the 8 warps in equal contiguous runs (a long row is shared by several warps, a warp rarely changes
        // row).  The i-th item of a warp goes through stage i mod RS of the warp's K/V ring.
        auto issue_item = [&](int item, int stage, int &sl) {      // sl: row-slot cursor, only moves forward
            while (item >= sh.cum[sl + 1]) ++sl;
            const int p0 = (item - sh.cum[sl]) * kFusedChunk;
            const int n_st = min(kFusedChunk, sh.lenst[sl] - p0);
            if (n_st > 0 && lane == 0) {
                uint64_t *bar = &sh.ring_bar[ww][stage];
                uint8_t *dst = ring + (static_cast<size_t>(ww) * RS + stage) * kRingStage;
                mbar_expect_tx(bar, n_st * 256);
                bulk_load(dst, sh.kptr[sl] + static_cast<size_t>(p0) * kHeadDim, n_st * 128, bar);
                bulk_load(dst + 2048, sh.vptr[sl] + static_cast<size_t>(p0) * kHeadDim, n_st * 128, bar);
            }
        };
        if (has_work) {
            load8(p.gamma + j * ks + cc * 8, gam);
            // fold constants of the output features this CTA finishes
            if (KIND == K_SELF) {
                if (pt < 192) {
                    const int col = (pt >> 6) * d + head * kHeadDim + (pt & 63);
                    sh.c1[pt] = p.c1[col];
                    sh.c2[pt] = p.c2[col];
                }
            } else if (KIND == K_CROSS) {
                if (pt < 64) { sh.c1[pt] = p.c1[head * kHeadDim + pt]; sh.c2[pt] = p.c2[head * kHeadDim + pt]; }
            } else {
                if (pt < 32) { sh.c1[pt] = p.c1[c * 128 + j * 32 + pt]; sh.c2[pt] = p.c2[c * 128 + j * 32 + pt]; }
            }
            if (KIND != K_FFN && ww == 0) {
                // row table of this CTA (static during the step) -> lengths, cache pointers, chunk prefix sums
                int len = 0;
                if (lane < SL) {
                    const int4 ri = p.row_info[2 * (j + kCS * lane) + parity];
                    const __nv_bfloat16 *kb = p.cache, *vb = p.cache;
                    int lst = 0;
                    if (ri.x >= 0) {
                        len = KIND == K_CROSS ? ri.z : ri.y + 1;
                        lst = KIND == K_CROSS ? len : len - 1;
                        if (KIND == K_CROSS) {
                            kb = p.cache + ((size_t)(0 * p.n_heads + head) * p.seq_capacity + ri.w) * kHeadDim;
                            vb = p.cache + ((size_t)(1 * p.n_heads + head) * p.seq_capacity + ri.w) * kHeadDim;
                        } else {
                            kb = p.cache + (((size_t)ri.x * 2 + 0) * p.n_heads + head) * (size_t)p.seq_capacity * kHeadDim;
                            vb = p.cache + (((size_t)ri.x * 2 + 1) * p.n_heads + head) * (size_t)p.seq_capacity * kHeadDim;
                        }
                    }
                    sh.kptr[lane] = kb; sh.vptr[lane] = vb; sh.len[lane] = len; sh.lenst[lane] = lst;
                }
                int chunks = (len + kFusedChunk - 1) / kFusedChunk;       // 0 for lanes without a row
                int incl = chunks;
#pragma unroll
                for (int o = 1; o < kMaxSlots; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                if (lane < kMaxSlots) sh.cum[lane + 1] = incl;
                if (lane == 0) sh.cum[0] = 0;
            }
        }
        worker_sync();                                     // fold constants and row table staged
        int item0 = 0, item1 = 0, sl_issue = 0, sl_use = 0;
        if (KIND != K_FFN && has_work) {
            const int n_items = sh.cum[SL], per = (n_items + 7) / 8;
            item0 = min(ww * per, n_items);
            item1 = min(item0 + per, n_items);
            // the first chunks of this warp are static data: they stream while the previous block still runs
            for (int i = 0; i < RS; ++i)
                if (item0 + i < item1) issue_item(item0 + i, i, sl_issue);
        }
        dep_wait();
        AED_TRACE_PUT(p.state, tcur, 50);          // dependency resolved
        const int n_rows = p.state->n_active;
        // local rows of this cluster that exist, and the step row of local row l
        const int n_loc = KIND == K_FFN ? min(n_rows, N) : min(max((n_rows - parity + 1) / 2, 0), N / 2);
        auto step_row = [&](int l) { return KIND == K_FFN ? l : 2 * l + parity; };
        bool ok = true;
        if (has_work) {
            // ---- 1. x slice -> statistics of the slice, gamma*x as bf16 planes -----------------------------------
            for (int ps0 = 0; ps0 * rows_per_pass < n_loc_cap; ps0 += 4) {
                float xv[4][8];
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int l = (ps0 + ps) * rows_per_pass + r_in_pass;
                    if (l < n_loc) load8_cg(p.x_in + (size_t)step_row(l) * d + j * ks + cc * 8, xv[ps]);
                    else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) xv[ps][e] = 0.f;
                    }
                }
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int l = (ps0 + ps) * rows_per_pass + r_in_pass;
                    if ((ps0 + ps) * rows_per_pass >= n_loc_cap) break;        // uniform over the block
                    float s = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) s += xv[ps][e];
                    s += __shfl_xor_sync(0xffffffffu, s, 1);
                    s += __shfl_xor_sync(0xffffffffu, s, 2);
                    s += __shfl_xor_sync(0xffffffffu, s, 4);
                    s += __shfl_xor_sync(0xffffffffu, s, 8);
                    if (cpr == 32) s += __shfl_xor_sync(0xffffffffu, s, 16);
                    const float mean = s / ks;
                    float q = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) { const float dv = xv[ps][e] - mean; q = fmaf(dv, dv, q); }
                    q += __shfl_xor_sync(0xffffffffu, q, 1);
                    q += __shfl_xor_sync(0xffffffffu, q, 2);
                    q += __shfl_xor_sync(0xffffffffu, q, 4);
                    q += __shfl_xor_sync(0xffffffffu, q, 8);
                    if (cpr == 32) q += __shfl_xor_sync(0xffffffffu, q, 16);
                    if (l < n_loc_cap) {
                        if (l < n_loc) {
                            if (KIND == K_FFN) {           // every CTA of the cluster needs every row's statistics
                                if (cc < kCS) st_cluster_f32x2(map_to_cta(stats_s, cc) + (j * kMaxRows + l) * 8, mean, q);
                            } else if (cc == 0) {          // the CTA that owns the row
                                st_cluster_f32x2(map_to_cta(stats_s, l & 3) + (j * kMaxRows + (l >> 2)) * 8, mean, q);
                            }
                        }
                        float y[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] = xv[ps][e] * gam[e];
                        uint4 hi, lo;
                        sg::split_planes(y, hi, lo);
                        const int kb = cc >> 3, ch = cc & 7;
                        uint8_t *tile = r2 + static_cast<size_t>(kb) * 2 * pb;
                        const int off = l * 128 + ((ch ^ (l & 7)) << 4);
                        *reinterpret_cast<uint4 *>(tile + off) = hi;
                        *reinterpret_cast<uint4 *>(tile + pb + off) = lo;
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bars.b)) : "memory");
            AED_TRACE_PUT(p.state, tcur, 51);      // operand planes written

            // ---- 3. partial sums of the first projection -> the CTA that finishes them ----------------------------
            ok = mbar_wait(&bars.d1, par, &sh.abort_flag);
            tc_fence_after_sync();
            AED_TRACE_PUT(p.state, tcur, 52);      // first projection complete
            if (ok) {
                const int acc = (KIND == K_SELF && ww >= 4) ? 1 : 0;
                const bool lanes_ok = KIND == K_SELF ? (acc == 0 || quarter < 2) : KIND == K_CROSS ? quarter < 2 : true;
                // two warps share a quarter of the lanes where one accumulator serves all 8 warps: split the columns
                const bool split_cols = KIND != K_SELF;
                const int col_lo = split_cols && ww >= 4 ? Nm / 2 : 0;
                const int col_hi = min(split_cols && ww < 4 ? Nm / 2 : Nm, n_loc);
                if (lanes_ok) {
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * Nm;
                    if (KIND == K_FFN) {
                        // lanes = 32 consecutive hidden features, all owned by CTA quarter
                        const uint32_t dst = map_to_cta(recv_s, quarter) + (static_cast<uint32_t>(j) * N * 32 + lane) * 4;
                        for (int c0 = (col_lo / 16) * 16; c0 < col_hi; c0 += 16) {
                            float v[16];
                            tmem_ld16(taddr + c0, v);
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                if (c0 + jj >= col_lo && c0 + jj < col_hi) st_cluster_f32(dst + (c0 + jj) * 128, v[jj]);
                        }
                    } else {
                        const int FE = KIND == K_SELF ? 192 : 64;
                        const int feat = (KIND == K_SELF && acc == 1 ? 128 : 0) + quarter * 32 + lane;
                        uint32_t peer[kCS];
#pragma unroll
                        for (int o = 0; o < kCS; ++o) peer[o] = map_to_cta(recv_s, o) + (static_cast<uint32_t>(j) * SL * FE + feat) * 4;
                        for (int c0 = (col_lo / 16) * 16; c0 < col_hi; c0 += 16) {
                            float v[16];
                            tmem_ld16(taddr + c0, v);
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) {
                                const int l = c0 + jj;                 // owner l & 3 = jj & 3, slot l >> 2
                                if (l >= col_lo && l < col_hi) st_cluster_f32(peer[jj & 3] + (l >> 2) * FE * 4, v[jj]);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane < kCS) arrive_remote(map_to_cta(cbar0_s, lane));     // first exchange, also on the abort path
            AED_TRACE_PUT(p.state, tcur, 53);      // partials sent
            ok = mbar_wait_cluster(&bars.c0, par, &sh.abort_flag) && ok;
            AED_TRACE_PUT(p.state, tcur, 54);      // first exchange complete

            if (KIND == K_FFN) {
                // ---- 4. hidden activations of this CTA's 32 features, written into every CTA's operand tile ------
                const int r = pt >> 2, c4 = pt & 3;
                if (ok && r < n_loc) {
                    float a[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) a[e] = 0.f;
#pragma unroll
                    for (int s = 0; s < kCS; ++s) {
                        float t8[8];
                        load8(recv + (static_cast<size_t>(s) * N + r) * 32 + c4 * 8, t8);
#pragma unroll
                        for (int e = 0; e < 8; ++e) a[e] += t8[e];
                    }
                    const float2 st = merge_stats(stats_recv + r, kMaxRows, ks, d, p.eps);
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        a[e] = fmaxf(fmaf(st.y, a[e] - st.x * sh.c1[c4 * 8 + e], sh.c2[c4 * 8 + e]), 0.f);
                    uint4 hi, lo;
                    sg::split_planes(a, hi, lo);
                    // k index inside the chunk: 32 j + 8 c4  ->  k-block j / 2, 16-byte chunk (j & 1) * 4 + c4
                    const int ch = (j & 1) * 4 + c4;
                    const uint32_t off = static_cast<uint32_t>(j >> 1) * 2 * pb + r * 128 + ((ch ^ (r & 7)) << 4);
#pragma unroll
                    for (int o = 0; o < kCS; ++o) {
                        const uint32_t dst = map_to_cta(r2_s, o) + off;
                        st_cluster_b128(dst, hi);
                        st_cluster_b128(dst + pb, lo);
                    }
                }
            } else {
                // ---- 4. attention for the rows of this CTA -------------------------------------------------------------
                const int FE = KIND == K_SELF ? 192 : 64;
                // 4a. warp s finishes the query (and the new key / value) of row slot s
                if (ok && ww < SL && sh.len[ww] > 0) {
                    const int sl = ww;
                    const float2 st = merge_stats(stats_recv + sl, kMaxRows, ks, d, p.eps);
                    float qv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) qv[e] = 0.f;
#pragma unroll
                    for (int s8 = 0; s8 < kCS; ++s8) {
                        float t8[8];
                        load8(recv + (static_cast<size_t>(s8) * SL + sl) * FE + dg * 8, t8);
#pragma unroll
                        for (int e = 0; e < 8; ++e) qv[e] += t8[e];
                    }
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        qv[e] = fmaf(st.y, qv[e] - st.x * sh.c1[dg * 8 + e], sh.c2[dg * 8 + e]) * p.scale;
                    if (pg == 0) {
                        *reinterpret_cast<float4 *>(sm_q + sl * kHeadDim + dg * 8) = make_float4(qv[0], qv[1], qv[2], qv[3]);
                        *reinterpret_cast<float4 *>(sm_q + sl * kHeadDim + dg * 8 + 4) = make_float4(qv[4], qv[5], qv[6], qv[7]);
                    }
                    if (KIND == K_SELF) {
                        float kn[8], vn[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) { kn[e] = 0.f; vn[e] = 0.f; }
#pragma unroll
                        for (int s8 = 0; s8 < kCS; ++s8) {
                            float t8[8];
                            const float *src = recv + (static_cast<size_t>(s8) * SL + sl) * FE + dg * 8;
                            load8(src + 64, t8);
#pragma unroll
                            for (int e = 0; e < 8; ++e) kn[e] += t8[e];
                            load8(src + 128, t8);
#pragma unroll
                            for (int e = 0; e < 8; ++e) vn[e] += t8[e];
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            kn[e] = fmaf(st.y, kn[e] - st.x * sh.c1[64 + dg * 8 + e], sh.c2[64 + dg * 8 + e]);
                            vn[e] = fmaf(st.y, vn[e] - st.x * sh.c1[128 + dg * 8 + e], sh.c2[128 + dg * 8 + e]);
                        }
                        Raw8<__nv_bfloat16> new_k, new_v;
                        new_k.set(kn);
                        new_v.set(vn);
                        if (pg == 0) {      // append to the cache (nobody reads this position during this launch) and keep a copy
                            const int pos = sh.len[sl] - 1;
                            new_k.store(const_cast<__nv_bfloat16 *>(sh.kptr[sl]) + (size_t)pos * kHeadDim + dg * 8);
                            new_v.store(const_cast<__nv_bfloat16 *>(sh.vptr[sl]) + (size_t)pos * kHeadDim + dg * 8);
                            new_k.store(sm_knew + sl * kHeadDim + dg * 8);
                            new_v.store(sm_vnew + sl * kHeadDim + dg * 8);
                        }
                    }
                }
                worker_sync();          // queries in place; the receive buffer is free for the partials
                AED_TRACE_PUT(p.state, tcur, 58);
                if (lane < SL) part[(ww * SL + lane) * kPartStride] = -INFINITY;
                __syncwarp();
                // 4b. this warp's chunks
                {
                    float m = -INFINITY, l = 0.f, acc8[8], qv[8];
                    int cur = -1;
                    auto flush = [&]() {
                        l += __shfl_xor_sync(0xffffffffu, l, 8);
                        l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            acc8[e] += __shfl_xor_sync(0xffffffffu, acc8[e], 8);
                            acc8[e] += __shfl_xor_sync(0xffffffffu, acc8[e], 16);
                        }
                        float *dst = part + (ww * SL + cur) * kPartStride;
                        if (lane == 0) { dst[0] = m; dst[1] = l; }
                        if (pg == 0) {
                            *reinterpret_cast<float4 *>(dst + 4 + dg * 8) = make_float4(acc8[0], acc8[1], acc8[2], acc8[3]);
                            *reinterpret_cast<float4 *>(dst + 8 + dg * 8) = make_float4(acc8[4], acc8[5], acc8[6], acc8[7]);
                        }
                    };
                    int i = 0;
                    for (int item = item0; item < item1 && ok; ++item, ++i) {
                        const int stage = i % RS;
                        while (item >= sh.cum[sl_use + 1]) ++sl_use;
                        const int sl = sl_use;
                        const int p0 = (item - sh.cum[sl]) * kFusedChunk;
                        const int len = sh.len[sl], len_st = sh.lenst[sl];
                        if (sl != cur) {
                            if (cur >= 0) flush();
                            cur = sl;
                            m = -INFINITY; l = 0.f;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc8[e] = 0.f;
                            load8(sm_q + sl * kHeadDim + dg * 8, qv);
                        }
                        AED_TRACE_PUT(p.state, tcur, 61);
                        if (len_st > p0) {                // a chunk that holds only the new position has no copy
                            ok = mbar_wait(&sh.ring_bar[ww][stage], (ring_phase >> stage) & 1u, &sh.abort_flag);
                            ring_phase ^= 1u << stage;
                        }
                        if (!ok) break;
                        AED_TRACE_PUT(p.state, tcur, 62);
                        const uint8_t *stg = ring + (static_cast<size_t>(ww) * RS + stage) * kRingStage;
                        Raw8<__nv_bfloat16> rk[4], rv[4];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const int pl = q4 * 4 + pg;                 // position inside the chunk
                            if (p0 + pl < len_st) {
                                rk[q4].load(reinterpret_cast<const __nv_bfloat16 *>(stg + pl * 128) + dg * 8);
                                rv[q4].load(reinterpret_cast<const __nv_bfloat16 *>(stg + 2048 + pl * 128) + dg * 8);
                            } else if (KIND == K_SELF && p0 + pl == len - 1) {
                                rk[q4].load(sm_knew + sl * kHeadDim + dg * 8);
                                rv[q4].load(sm_vnew + sl * kHeadDim + dg * 8);
                            } else { rk[q4].zero(); rv[q4].zero(); }
                        }
                        __syncwarp();                                  // the stage has been read: refill it
                        AED_TRACE_PUT(p.state, tcur, 63);
                        if (item + RS < item1) issue_item(item + RS, stage, sl_issue);
                        AED_TRACE_PUT(p.state, tcur, 64);
                        float s4[4], cmax = -INFINITY;
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            float kf[8], dot = 0.f;
                            rk[q4].get(kf);
#pragma unroll
                            for (int e = 0; e < 8; ++e) dot = fmaf(qv[e], kf[e], dot);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                            s4[q4] = (p0 + q4 * 4 + pg < len) ? dot : -INFINITY;
                            cmax = fmaxf(cmax, s4[q4]);
                        }
                        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
                        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));      // finite: the chunk has a position
                        const float m_new = fmaxf(m, cmax);
                        const float corr = expf(m - m_new);
                        l *= corr;
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc8[e] *= corr;
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float pr = expf(s4[q4] - m_new);
                            float vf[8];
                            rv[q4].get(vf);
                            l += pr;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc8[e] = fmaf(pr, vf[e], acc8[e]);
                        }
                        m = m_new;
                        AED_TRACE_PUT(p.state, tcur, 65);
                    }
                    if (cur >= 0 && ok) flush();
                }
                AED_TRACE_PUT(p.state, tcur, 59);
                worker_sync();
                AED_TRACE_PUT(p.state, tcur, 60);
                // 4c. warp s merges the partials of row slot s and sends the result to every CTA's operand tile;
                //     lane group pg writes to CTA pg
                if (ok && ww < SL && sh.len[ww] > 0) {
                    const int sl = ww, r_att = j + kCS * sl;      // local row = row of the operand tile
                    float big = -INFINITY;
#pragma unroll
                    for (int w8 = 0; w8 < 8; ++w8) big = fmaxf(big, part[(w8 * SL + sl) * kPartStride]);
                    float lsum = 0.f, o[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] = 0.f;
#pragma unroll
                    for (int w8 = 0; w8 < 8; ++w8) {
                        const float *src = part + (w8 * SL + sl) * kPartStride;
                        const float mw = src[0];
                        if (mw == -INFINITY) continue;             // uniform over the warp
                        const float wgt = expf(mw - big);
                        lsum = fmaf(src[1], wgt, lsum);
                        float a8[8];
                        load8(src + 4 + dg * 8, a8);
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] = fmaf(a8[e], wgt, o[e]);
                    }
                    const float inv = 1.f / lsum;
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] *= inv;
                    uint4 hi, lo;
                    sg::split_planes(o, hi, lo);
                    const uint32_t off = r_att * 128 + ((dg ^ (r_att & 7)) << 4);
                    const uint32_t dst = map_to_cta(ap_s, pg) + off;
                    st_cluster_b128(dst, hi);
                    st_cluster_b128(dst + pb, lo);
                }
            }
            fence_async_proxy();
            __syncwarp();
            if (lane < kCS) arrive_remote(map_to_cta(cbar1_s, lane));     // second exchange
            AED_TRACE_PUT(p.state, tcur, 55);      // attention / activation done

            // ---- 5. second projection: partial over this head / chunk, added into x_out -----------------------------
            // The residual x_in and the bias are one more term of the sum: among the clusters that share this
            // cluster's rows, the one whose head / chunk index equals l mod n_work adds them for local row l, while
            // the MMAs of the second projection run.  All additions are 16-byte reductions.
            const int g4n = of / 4;                            // groups of 4 features per row
            {
                const int who = KIND == K_FFN ? c : head;
                const int n_res = n_loc > who ? (n_loc - who + n_work - 1) / n_work : 0;      // local rows who, who + n_work, ...
                for (int idx = pt; idx < n_res * g4n; idx += 256) {
                    const int r = step_row(who + n_work * (idx / g4n)), f4 = (idx % g4n) * 4;
                    float4 v = __ldcg(reinterpret_cast<const float4 *>(p.x_in + (size_t)r * d + j * of + f4));
                    if (p.bias2) {
                        float b4[4];
                        load4(p.bias2 + j * of + f4, b4);
                        v.x += b4[0]; v.y += b4[1]; v.z += b4[2]; v.w += b4[3];
                    }
                    sg::red_add_v4(p.x_out + (size_t)r * d + j * of + f4, v);
                }
            }
            ok = mbar_wait(&bars.d2, par, &sh.abort_flag) && ok;
            tc_fence_after_sync();
            AED_TRACE_PUT(p.state, tcur, 56);      // second projection complete
            // accumulators [feature lane][local row] -> shared memory [local row][feature]; the operand planes (and,
            // in the FFN block, the receive buffer in front of them) are free now
            float *trans = KIND == K_FFN ? recv : reinterpret_cast<float *>(r2);
            const int pitch = of + 4;
            {
                const int m = mt2 == 2 ? (ww >> 2) : 0;        // 128-feature tile of this warp
                const int f = m * kTileM + quarter * 32 + lane;
                const int col_lo = mt2 == 2 || ww < 4 ? 0 : Nm / 2;
                const int col_hi = min(mt2 == 2 || ww >= 4 ? Nm : Nm / 2, n_loc);
                if (ok) {
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + (2 + m) * Nm;
                    for (int c0 = (col_lo / 16) * 16; c0 < col_hi; c0 += 16) {
                        float v[16];
                        tmem_ld16(taddr + c0, v);
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const int l = c0 + jj;
                            if (l >= col_lo && l < col_hi) trans[l * pitch + f] = v[jj];
                        }
                    }
                }
            }
            worker_sync();
            if (ok) {
                for (int idx = pt; idx < n_loc * g4n; idx += 256) {
                    const int l = idx / g4n, f4 = (idx % g4n) * 4;
                    const float4 v = *reinterpret_cast<const float4 *>(trans + l * pitch + f4);
                    sg::red_add_v4(p.x_out + (size_t)step_row(l) * d + j * of + f4, v);
                }
            }
            AED_TRACE_PUT(p.state, tcur, 57);              // reductions issued
        }
    }
}

// One block per launch, chained with programmatic dependent launch.  grid: 128 CTAs = 32 clusters of 4.
// map_w1 / map_w2: weight matrices of the first and second projection, boxes of 64 rows x 64 k.
template <int KIND>
__global__ void __launch_bounds__(kClThreads, 1)
cluster_block_kernel(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2, ClusterParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(16) CtaShared sh;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) init_cta_shared(sh);
    if (warp == 1) tmem_alloc(&sh.tmem_slot, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_slot;
    cluster_sync_all();                              // every CTA of the cluster has its barriers in place
    sg::pdl_launch_dependents();
    uint32_t ring_phase = 0;
    run_block<KIND, false>(p, &map_w1, &map_w2, p.n_tile, 0u, sh, smem_dyn, tmem_base, ring_phase, nullptr, 0);
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                              // nobody writes into a CTA that has left
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(&p.state->error, kErrTimeout);
}

// All blocks of a step in one launch: blocks[3 l + k] describes block k of layer l, maps[6 l + 2 k] and
// maps[6 l + 2 k + 1] are its weight matrices.  Between two blocks every CTA adds one to the arrival counter
// (DecState::grid_sync, cleared by the first kernel of the step) and the next block reads x_in once all CTAs of the
// grid have arrived; static data of the next block (weights, cached keys and values) is requested before that.
// All 128 CTAs must be resident at once (checked by the host with the occupancy query).
__global__ void __launch_bounds__(kClThreads, 1)
cluster_step_kernel(const ClusterParams *__restrict__ blocks, const CUtensorMap *__restrict__ maps, int n_blocks, int n_tile)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(16) CtaShared sh;
    __shared__ __align__(16) ClusterParams sp[2];
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) init_cta_shared(sh);
    if (warp == 1) tmem_alloc(&sh.tmem_slot, kTmemCols);
    constexpr int kWords = sizeof(ClusterParams) / 4;
    if (threadIdx.x >= 320 && threadIdx.x - 320 < kWords)
        reinterpret_cast<int *>(&sp[0])[threadIdx.x - 320] = reinterpret_cast<const int *>(&blocks[0])[threadIdx.x - 320];
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_slot;
    cluster_sync_all();
    uint32_t ring_phase = 0;
    DecState *state = sp[0].state;
    for (int b = 0; b < n_blocks; ++b) {
        const ClusterParams &p = sp[b & 1];
        const int kind = b % 3, layer = b / 3;
        const CUtensorMap *m1 = maps + 6 * layer + 2 * kind, *m2 = m1 + 1;
        const uint32_t par = layer & 1;
        const int target = b * static_cast<int>(gridDim.x);
        // the description of the next block travels while this one runs
        if (b + 1 < n_blocks && threadIdx.x >= 320 && threadIdx.x - 320 < kWords)
            reinterpret_cast<int *>(&sp[(b + 1) & 1])[threadIdx.x - 320] =
                reinterpret_cast<const int *>(&blocks[b + 1])[threadIdx.x - 320];
        if (kind == K_SELF) run_block<K_SELF, true>(p, m1, m2, n_tile, par, sh, smem_dyn, tmem_base, ring_phase, &state->grid_sync, target);
        else if (kind == K_CROSS) run_block<K_CROSS, true>(p, m1, m2, n_tile, par, sh, smem_dyn, tmem_base, ring_phase, &state->grid_sync, target);
        else run_block<K_FFN, true>(p, m1, m2, n_tile, par, sh, smem_dyn, tmem_base, ring_phase, &state->grid_sync, target);
        // end of the block: this CTA's shared memory and accumulators are free again, its additions to x_out are
        // ordered before its arrival
        fence_async_proxy();                         // generic writes to shared memory before the next block's TMA
        tc_fence_before_sync();
        __syncthreads();
        cluster_sync_all();
        tc_fence_after_sync();
        if (threadIdx.x == 0 && b + 1 < n_blocks) {
            __threadfence();
            atomicAdd(&state->grid_sync, 1);
        }
    }
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(&state->error, kErrTimeout);
}

}  // namespace cl
}  // namespace aed
