// Head-parallel decode step for small batches (at most 64 rows): three cluster kernels per layer.
//
// A decoder layer has three places where every output needs the whole residual row x: before the self-attention
// projections (LN1), before the cross-attention query projection (LN2) and before the feed-forward network (LN3).
// Everything between two such places can be split over attention heads (or over slices of the FFN hidden layer)
// without any exchange between the parts, so a layer is run as three "blocks":
//
//   K_SELF   x_out = x_in + Wo  . selfattn (LN1(x_in))      cluster c = head c
//   K_CROSS  x_out = x_in + Woc . crossattn(LN2(x_in))      cluster c = head c
//   K_FFN    x_out = x_in + W2 . relu(W1 . LN3(x_in) + b1) + b2      cluster c = hidden features 256c .. 256c+255
//
// Each block is one launch of 16 clusters of 8 CTAs.  Inside a cluster the 8 CTAs split the contraction dimension
// of the first projection (K = d_model, d/8 columns each) and the output features of the second one (d/8 each);
// partial results travel through distributed shared memory:
//
//   1. every CTA loads its d/8 columns of x_in for all rows, folds the LayerNorm scale in (gamma*x, bf16 high and
//      low planes) and computes the (mean, M2) of its slice of every row;
//   2. tcgen05.mma: partial[feature, row] over the CTA's K slice (weights are the A operand, fetched by TMA before
//      the dependency wait because they are static);
//   3. the partials are scattered to the CTA that owns the row (attention blocks: row r belongs to CTA r mod 8) or
//      the hidden feature (FFN: 32 features per CTA), together with the slice statistics; an mbarrier with
//      cluster-scope release/acquire marks the end of the exchange;
//   4. the owner sums the 8 partials, finishes the LayerNorm (rstd*(raw - mean*c1) + c2, see step_gemm.cuh) and
//      runs attention for its rows over the ragged cache (or applies ReLU), then writes the result as bf16 planes
//      straight into the B-operand tile of all 8 CTAs;
//   5. tcgen05.mma of the second projection over the head's 64 (or the chunk's 256) input features, d/8 output
//      features per CTA, and red.global.add of the partial into x_out, which was cleared by an earlier block.
//
// x rotates through three buffers (read, accumulate, clear) so that a fast cluster can never add into rows that a
// slow cluster of the same launch still reads.  Only the sum over heads / hidden chunks goes through global
// memory: three exchanges per layer instead of eight.
//
// Every wait is bounded; a CTA that gives up still performs all its cluster arrivals, so that its peers do not
// wait for it, and raises the error word of the decode state.
#pragma once
#include "step_gemm.cuh"
#include "step_kernels.cuh"

namespace aed {
namespace cl {

using namespace tc;

constexpr int kCS = 8;               // CTAs per cluster
constexpr int kClusters = 16;
constexpr int kClThreads = 384;      // warp 0 TMA, warp 1 MMA, warps 2..9 workers, warps 10..11 side jobs
constexpr int kSlot = 16384;         // one weight tile: 128 rows x 64 k, bf16
constexpr int kMaxTiles = 8;
constexpr int kMaxRows = 64;
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
    int n_slots, w_off, recv_off, r2_off, ap_off, stats_off, total;
};

// Dynamic shared memory of one block kind: weight slots | receive buffer | operand planes | attention planes | stats
__host__ __device__ inline ClSmem cl_layout(int kind, int n_tile, int kbs)
{
    ClSmem s;
    const int tiles = kind == K_SELF ? 2 * kbs + 1 : kind == K_CROSS ? kbs + 1 : 2 * kbs + 4;
    s.n_slots = tiles < 5 ? tiles : 5;
    const int recv = kind == K_SELF ? n_tile * 768 : kind == K_CROSS ? n_tile * 256 : n_tile * 1024;
    const int r2 = kind == K_FFN ? n_tile * 1024 : kbs * 2 * n_tile * 128;
    const int ap = kind == K_FFN ? 0 : 2 * n_tile * 128;
    s.w_off = 0;
    s.recv_off = s.w_off + s.n_slots * kSlot;
    s.r2_off = s.recv_off + recv;
    s.ap_off = s.r2_off + r2;
    s.stats_off = s.ap_off + ap;
    s.total = s.stats_off + kCS * kMaxRows * 8;
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
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// (mean, rstd) of a row from the (mean, M2) of its 8 equally long slices
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

// grid: 128 CTAs = 16 clusters of 8.  map_w1 / map_w2: weight matrices of the first and second projection,
// boxes of 64 rows x 64 k.
template <int KIND>
__global__ void __launch_bounds__(kClThreads, 1)
cluster_block_kernel(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2, ClusterParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_w[kMaxTiles];     // one per weight tile, each used once
    __shared__ __align__(8) uint64_t bar_b, bar_d1, bar_d2, cbar0, cbar1;   // cbar0 / cbar1: first / second exchange of the cluster
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float sm_c1[192], sm_c2[192];
    __shared__ float sm_m[8], sm_l[8];
    __shared__ __align__(16) float sm_acc[8][kHeadDim];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = static_cast<int>(cluster_ctarank());
    const int c = static_cast<int>(cluster_index());
    const int d = p.d, ks = d / kCS, kbs = ks / kBlockK, of = ks;
    const int N = p.n_tile;
    const int n_work = KIND == K_FFN ? p.d_ffn / 256 : p.n_heads;      // clusters that have a head / hidden chunk
    const bool has_work = c < n_work;
    const ClSmem lay = cl_layout(KIND, N, kbs);
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *w_slots = base + lay.w_off;
    float *recv = reinterpret_cast<float *>(base + lay.recv_off);
    uint8_t *r2 = base + lay.r2_off;                 // x planes; K_FFN: later the hidden planes
    uint8_t *ap = base + lay.ap_off;                 // attention output planes
    float2 *stats_recv = reinterpret_cast<float2 *>(base + lay.stats_off);
    const int pb = N * 128;                          // bytes of one plane of one k-block
    const int n_tiles1 = KIND == K_SELF ? 2 * kbs : KIND == K_CROSS ? kbs : 2 * kbs;
    const int n_tiles2 = KIND == K_FFN ? 4 : 1;
    const int n_tiles = n_tiles1 + n_tiles2;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kMaxTiles; ++i) mbar_init(&bar_w[i], 1);
        mbar_init(&bar_b, 8);
        mbar_init(&bar_d1, 1);
        mbar_init(&bar_d2, 1);
        mbar_init(&cbar0, kCS * 8);                  // 8 worker warps of each of the 8 CTAs
        mbar_init(&cbar1, kCS * 8);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_slot, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    cluster_sync_all();                              // every CTA of the cluster has its barriers in place
    sg::pdl_launch_dependents();
    AED_TRACE_BEGIN(p.state, 24 + KIND);

    if (warp == 0) {
        // ---- weight tiles by TMA: static data, requested before the dependency wait ---------------------------
        if (lane == 0 && has_work) {
            prefetch_tensormap(&map_w1);
            prefetch_tensormap(&map_w2);
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                if (t >= lay.n_slots) {              // K_FFN: the slot held a tile of the first projection
                    ok = mbar_wait(&bar_d1, 0, &abort_flag);
                    if (!ok) break;
                }
                uint8_t *slot = w_slots + static_cast<size_t>(t % lay.n_slots) * kSlot;
                if (t < n_tiles1) {
                    const int kb = KIND == K_SELF ? t >> 1 : KIND == K_CROSS ? t : t % kbs;
                    const int kc = j * ks + kb * kBlockK;
                    if (KIND == K_SELF) {
                        if ((t & 1) == 0) {          // query rows | key rows of head c
                            mbar_expect_tx(&bar_w[t], 2 * 8192);
                            tma_load_2d(slot, &map_w1, kc, c * kHeadDim, &bar_w[t]);
                            tma_load_2d(slot + 8192, &map_w1, kc, d + c * kHeadDim, &bar_w[t]);
                        } else {                     // value rows
                            mbar_expect_tx(&bar_w[t], 8192);
                            tma_load_2d(slot, &map_w1, kc, 2 * d + c * kHeadDim, &bar_w[t]);
                        }
                    } else if (KIND == K_CROSS) {
                        mbar_expect_tx(&bar_w[t], 8192);
                        tma_load_2d(slot, &map_w1, kc, c * kHeadDim, &bar_w[t]);
                    } else {                         // 128 hidden features of chunk c
                        const int mt = t / kbs;
                        mbar_expect_tx(&bar_w[t], 2 * 8192);
                        tma_load_2d(slot, &map_w1, kc, c * 256 + mt * 128, &bar_w[t]);
                        tma_load_2d(slot + 8192, &map_w1, kc, c * 256 + mt * 128 + 64, &bar_w[t]);
                    }
                } else {                             // second projection: this CTA's d/8 output features
                    const int q = t - n_tiles1;
                    const int kc = KIND == K_FFN ? c * 256 + q * kBlockK : c * kHeadDim;
                    mbar_expect_tx(&bar_w[t], of * 128);
                    for (int b = 0; b < of / 64; ++b) tma_load_2d(slot + b * 8192, &map_w2, kc, j * of + b * 64, &bar_w[t]);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue --------------------------------------------------------------------------------------------
        if (lane == 0 && has_work) {
            const uint32_t idesc = instr_desc_bf16(N);
            bool ok = mbar_wait(&bar_b, 0, &abort_flag);
            for (int t = 0; t < n_tiles1 && ok; ++t) {
                ok = mbar_wait(&bar_w[t], 0, &abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const int kb = KIND == K_SELF ? t >> 1 : KIND == K_CROSS ? t : t % kbs;
                const int acc = KIND == K_SELF ? (t & 1) : KIND == K_CROSS ? 0 : t / kbs;
                const uint32_t sa = smem_u32(w_slots + static_cast<size_t>(t % lay.n_slots) * kSlot);
                const uint32_t sb = smem_u32(r2 + static_cast<size_t>(kb) * 2 * pb);
                const uint64_t da = smem_desc_sw128(sa), dh = smem_desc_sw128(sb), dl = smem_desc_sw128(sb + pb);
                const uint32_t td = tmem_base + acc * N;
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dh + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dl + 2 * k, idesc, 1u);
            }
            if (ok) mma_commit(&bar_d1);
            // second projection: its B operand is complete when the second exchange of the cluster is
            ok = ok && mbar_wait_cluster(&cbar1, 0, &abort_flag);
            if (ok) {
                fence_async_proxy();
                tc_fence_after_sync();
                const uint32_t td = tmem_base + 2 * N;
                for (int q = 0; q < n_tiles2 && ok; ++q) {
                    const int t = n_tiles1 + q;
                    ok = mbar_wait(&bar_w[t], 0, &abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(w_slots + static_cast<size_t>(t % lay.n_slots) * kSlot);
                    const uint32_t sb = smem_u32(KIND == K_FFN ? r2 + static_cast<size_t>(q) * 2 * pb : ap);
                    const uint64_t da = smem_desc_sw128(sa), dh = smem_desc_sw128(sb), dl = smem_desc_sw128(sb + pb);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dh + 2 * k, idesc, (q > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(td, da + 2 * k, dl + 2 * k, idesc, 1u);
                }
                if (ok) mma_commit(&bar_d2);
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
        if (p.pf_cache && c < p.n_heads) {
            // keys and values that this CTA's rows read in the next attention block: thread = (row slot, k|v)
            const int slot = st >> 1, kv = st & 1;
            if (slot < N / kCS) {
                const int4 ri = p.row_info[j + kCS * slot];
                if (ri.x >= 0) {
                    const __nv_bfloat16 *src;
                    int len;
                    if (p.pf_cross) {
                        src = p.pf_cache + ((size_t)(kv * p.n_heads + c) * p.pf_capacity + ri.w) * kHeadDim;
                        len = ri.z;
                    } else {
                        src = p.pf_cache + (((size_t)ri.x * 2 + kv) * p.n_heads + c) * (size_t)p.pf_capacity * kHeadDim;
                        len = ri.y;
                    }
                    for (int off = 0; off < len; off += 32) {
                        const int rows = min(32, len - off);
                        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + (size_t)off * kHeadDim), "r"(rows * 128) : "memory");
                    }
                }
            }
        }
        sg::pdl_wait();
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
        const uint32_t recv_s = smem_u32(recv), stats_s = smem_u32(stats_recv);
        const uint32_t cbar0_s = smem_u32(&cbar0), cbar1_s = smem_u32(&cbar1);
        const uint32_t ap_s = smem_u32(ap), r2_s = smem_u32(r2);
        // x slice geometry: thread = (row within pass, 8-column chunk cc)
        const int cpr = ks >> 3, rows_per_pass = 256 / cpr;
        const int cc = pt % cpr, r_in_pass = pt / cpr;
        const int SL = N / kCS;                            // row slots per CTA in the attention blocks
        // attention geometry: G warps per row slot
        const int G = 8 / (SL < 1 ? 1 : SL);
        const int slot = ww / G, g = ww % G;
        const int r_att = j + kCS * slot;
        const int dg = lane & 7, pg = lane >> 3;
        int4 ri = make_int4(-1, 0, 0, 0);
        const __nv_bfloat16 *kbase = nullptr, *vbase = nullptr;
        int len = 0, len_static = 0;
        Raw8<__nv_bfloat16> rk[4], rv[4];
        float gam[8];
        if (has_work) {
            load8(p.gamma + j * ks + cc * 8, gam);
            // fold constants of the output features this CTA finishes
            if (KIND == K_SELF) {
                if (pt < 192) {
                    const int col = (pt >> 6) * d + c * kHeadDim + (pt & 63);
                    sm_c1[pt] = p.c1[col];
                    sm_c2[pt] = p.c2[col];
                }
            } else if (KIND == K_CROSS) {
                if (pt < 64) { sm_c1[pt] = p.c1[c * kHeadDim + pt]; sm_c2[pt] = p.c2[c * kHeadDim + pt]; }
            } else {
                if (pt < 32) { sm_c1[pt] = p.c1[c * 256 + j * 32 + pt]; sm_c2[pt] = p.c2[c * 256 + j * 32 + pt]; }
            }
            if (KIND != K_FFN) {
                ri = p.row_info[r_att];
                if (ri.x >= 0) {
                    len = KIND == K_CROSS ? ri.z : ri.y + 1;
                    len_static = KIND == K_CROSS ? len : len - 1;
                    if (KIND == K_CROSS) {
                        kbase = p.cache + ((size_t)(0 * p.n_heads + c) * p.seq_capacity + ri.w) * kHeadDim;
                        vbase = p.cache + ((size_t)(1 * p.n_heads + c) * p.seq_capacity + ri.w) * kHeadDim;
                    } else {
                        kbase = p.cache + (((size_t)ri.x * 2 + 0) * p.n_heads + c) * (size_t)p.seq_capacity * kHeadDim;
                        vbase = p.cache + (((size_t)ri.x * 2 + 1) * p.n_heads + c) * (size_t)p.seq_capacity * kHeadDim;
                    }
                    // first chunk of this warp: static positions, streamed while the previous block still runs
                    const int p0 = g * kFusedChunk;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int pos = p0 + i * 4 + pg;
                        if (pos < len_static) {
                            rk[i].load(kbase + (size_t)pos * kHeadDim + dg * 8);
                            rv[i].load(vbase + (size_t)pos * kHeadDim + dg * 8);
                        } else { rk[i].zero(); rv[i].zero(); }
                    }
                }
            }
        }
        worker_sync();                                     // fold constants staged
        sg::pdl_wait();
        const int n_rows = p.state->n_active;
        bool ok = true;
        if (has_work) {
            // ---- 1. x slice -> statistics of the slice, gamma*x as bf16 planes -----------------------------------
            float xv[4][8];
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const int r = ps * rows_per_pass + r_in_pass;
                if (r < N && r < n_rows) load8(p.x_in + (size_t)r * d + j * ks + cc * 8, xv[ps]);
                else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) xv[ps][e] = 0.f;
                }
            }
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const int r = ps * rows_per_pass + r_in_pass;
                if (ps * rows_per_pass >= N) break;        // uniform over the block
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) s += xv[ps][e];
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                s += __shfl_xor_sync(0xffffffffu, s, 2);
                s += __shfl_xor_sync(0xffffffffu, s, 4);
                if (cpr == 16) s += __shfl_xor_sync(0xffffffffu, s, 8);
                const float mean = s / ks;
                float q = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) { const float dv = xv[ps][e] - mean; q = fmaf(dv, dv, q); }
                q += __shfl_xor_sync(0xffffffffu, q, 1);
                q += __shfl_xor_sync(0xffffffffu, q, 2);
                q += __shfl_xor_sync(0xffffffffu, q, 4);
                if (cpr == 16) q += __shfl_xor_sync(0xffffffffu, q, 8);
                if (r < N) {
                    if (r < n_rows) {
                        if (KIND == K_FFN) {               // every CTA of the cluster needs every row's statistics
                            if (cc < kCS) st_cluster_f32x2(map_to_cta(stats_s, cc) + (j * kMaxRows + r) * 8, mean, q);
                        } else if (cc == 0) {              // the CTA that owns the row
                            st_cluster_f32x2(map_to_cta(stats_s, r & 7) + (j * kMaxRows + (r >> 3)) * 8, mean, q);
                        }
                    }
                    float y[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) y[e] = xv[ps][e] * gam[e];
                    uint4 hi, lo;
                    sg::split_planes(y, hi, lo);
                    const int kb = cc >> 3, ch = cc & 7;
                    uint8_t *tile = r2 + static_cast<size_t>(kb) * 2 * pb;
                    const int off = r * 128 + ((ch ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4 *>(tile + off) = hi;
                    *reinterpret_cast<uint4 *>(tile + pb + off) = lo;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_b)) : "memory");

            // ---- 3. partial sums of the first projection -> the CTA that finishes them ----------------------------
            ok = mbar_wait(&bar_d1, 0, &abort_flag);
            tc_fence_after_sync();
            if (ok) {
                const int acc = (KIND == K_CROSS) ? 0 : (ww < 4 ? 0 : 1);
                const bool lanes_ok = KIND == K_SELF ? (acc == 0 || quarter < 2) : KIND == K_CROSS ? quarter < 2 : true;
                const int col_lo = KIND == K_CROSS ? (ww < 4 ? 0 : N / 2) : 0;
                const int col_hi = KIND == K_CROSS ? (ww < 4 ? N / 2 : N) : N;
                if (lanes_ok) {
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * N;
                    if (KIND == K_FFN) {
                        // lanes = 32 consecutive hidden features, all owned by CTA acc*4 + quarter
                        const uint32_t dst = map_to_cta(recv_s, acc * 4 + quarter) + (static_cast<uint32_t>(j) * N * 32 + lane) * 4;
                        for (int c0 = 0; c0 < N; c0 += 16) {
                            float v[16];
                            tmem_ld16(taddr + c0, v);
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                if (c0 + jj < n_rows) st_cluster_f32(dst + (c0 + jj) * 128, v[jj]);
                        }
                    } else {
                        const int FE = KIND == K_SELF ? 192 : 64;
                        const int feat = (KIND == K_SELF && acc == 1 ? 128 : 0) + quarter * 32 + lane;
                        uint32_t peer[kCS];
#pragma unroll
                        for (int o = 0; o < kCS; ++o) peer[o] = map_to_cta(recv_s, o) + (static_cast<uint32_t>(j) * SL * FE + feat) * 4;
                        for (int c0 = 0; c0 < N; c0 += 16) {
                            float v[16];
                            tmem_ld16(taddr + c0, v);
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) {
                                const int r = c0 + jj;                 // owner r & 7 = jj & 7, slot r >> 3
                                if (r >= col_lo && r < col_hi && r < n_rows) st_cluster_f32(peer[jj & 7] + (r >> 3) * FE * 4, v[jj]);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane < kCS) arrive_remote(map_to_cta(cbar0_s, lane));     // first exchange, also on the abort path
            ok = mbar_wait_cluster(&cbar0, 0, &abort_flag) && ok;

            if (KIND == K_FFN) {
                // ---- 4. hidden activations of this CTA's 32 features, written into every CTA's operand tile ------
                const int r = pt >> 2, c4 = pt & 3;
                if (ok && r < N && r < n_rows) {
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
                        a[e] = fmaxf(fmaf(st.y, a[e] - st.x * sm_c1[c4 * 8 + e], sm_c2[c4 * 8 + e]), 0.f);
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
                float m = -INFINITY, l = 0.f, acc8[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc8[e] = 0.f;
                const bool row_ok = ok && ri.x >= 0 && r_att < n_rows;
                if (row_ok) {
                    const int FE = KIND == K_SELF ? 192 : 64;
                    const float2 st = merge_stats(stats_recv + slot, kMaxRows, ks, d, p.eps);
                    float qv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) qv[e] = 0.f;
#pragma unroll
                    for (int s = 0; s < kCS; ++s) {
                        float t8[8];
                        load8(recv + (static_cast<size_t>(s) * SL + slot) * FE + dg * 8, t8);
#pragma unroll
                        for (int e = 0; e < 8; ++e) qv[e] += t8[e];
                    }
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        qv[e] = fmaf(st.y, qv[e] - st.x * sm_c1[dg * 8 + e], sm_c2[dg * 8 + e]) * p.scale;
                    const int new_chunk = (len - 1) / kFusedChunk;
                    const bool owns_new = KIND == K_SELF && g == new_chunk % G;
                    Raw8<__nv_bfloat16> new_k, new_v;
                    if (owns_new) {
                        float kn[8], vn[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) { kn[e] = 0.f; vn[e] = 0.f; }
#pragma unroll
                        for (int s = 0; s < kCS; ++s) {
                            float t8[8];
                            const float *src = recv + (static_cast<size_t>(s) * SL + slot) * FE + dg * 8;
                            load8(src + 64, t8);
#pragma unroll
                            for (int e = 0; e < 8; ++e) kn[e] += t8[e];
                            load8(src + 128, t8);
#pragma unroll
                            for (int e = 0; e < 8; ++e) vn[e] += t8[e];
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            kn[e] = fmaf(st.y, kn[e] - st.x * sm_c1[64 + dg * 8 + e], sm_c2[64 + dg * 8 + e]);
                            vn[e] = fmaf(st.y, vn[e] - st.x * sm_c1[128 + dg * 8 + e], sm_c2[128 + dg * 8 + e]);
                        }
                        new_k.set(kn);
                        new_v.set(vn);
                        if (pg == 0) {      // append; nobody else reads this position during this launch
                            new_k.store(const_cast<__nv_bfloat16 *>(kbase) + (size_t)(len - 1) * kHeadDim + dg * 8);
                            new_v.store(const_cast<__nv_bfloat16 *>(vbase) + (size_t)(len - 1) * kHeadDim + dg * 8);
                        }
                    }
                    bool loaded = true;
                    for (int p0 = g * kFusedChunk; p0 < len; p0 += G * kFusedChunk) {
                        if (!loaded) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int pos = p0 + i * 4 + pg;
                                if (pos < len_static) {
                                    rk[i].load(kbase + (size_t)pos * kHeadDim + dg * 8);
                                    rv[i].load(vbase + (size_t)pos * kHeadDim + dg * 8);
                                } else { rk[i].zero(); rv[i].zero(); }
                            }
                        }
                        loaded = false;
                        if (owns_new && p0 == new_chunk * kFusedChunk) {
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                if (p0 + i * 4 + pg == len - 1) { rk[i] = new_k; rv[i] = new_v; }
                        }
                        float s4[4], cmax = -INFINITY;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float kf[8], dot = 0.f;
                            rk[i].get(kf);
#pragma unroll
                            for (int e = 0; e < 8; ++e) dot = fmaf(qv[e], kf[e], dot);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                            dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                            s4[i] = (p0 + i * 4 + pg < len) ? dot : -INFINITY;
                            cmax = fmaxf(cmax, s4[i]);
                        }
                        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
                        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
                        const float m_new = fmaxf(m, cmax);
                        const float corr = expf(m - m_new);
                        l *= corr;
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc8[e] *= corr;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float pr = expf(s4[i] - m_new);
                            float vf[8];
                            rv[i].get(vf);
                            l += pr;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc8[e] = fmaf(pr, vf[e], acc8[e]);
                        }
                        m = m_new;
                    }
                    l += __shfl_xor_sync(0xffffffffu, l, 8);
                    l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        acc8[e] += __shfl_xor_sync(0xffffffffu, acc8[e], 8);
                        acc8[e] += __shfl_xor_sync(0xffffffffu, acc8[e], 16);
                    }
                }
                if (lane == 0) { sm_m[ww] = m; sm_l[ww] = l; }
                if (pg == 0) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) sm_acc[ww][dg * 8 + e] = acc8[e];
                }
                worker_sync();
                if (row_ok && g == 0) {
                    // merge the G warps of the row; lane group pg sends to CTAs 2 pg and 2 pg + 1
                    float big = -INFINITY;
                    for (int w = 0; w < G; ++w) big = fmaxf(big, sm_m[slot * G + w]);
                    float lsum = 0.f, o[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] = 0.f;
                    for (int w = 0; w < G; ++w) {
                        const float mw = sm_m[slot * G + w];
                        const float wgt = (mw == -INFINITY) ? 0.f : expf(mw - big);
                        lsum = fmaf(sm_l[slot * G + w], wgt, lsum);
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] = fmaf(sm_acc[slot * G + w][dg * 8 + e], wgt, o[e]);
                    }
                    const float inv = 1.f / lsum;
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] *= inv;
                    uint4 hi, lo;
                    sg::split_planes(o, hi, lo);
                    const uint32_t off = r_att * 128 + ((dg ^ (r_att & 7)) << 4);
#pragma unroll
                    for (int o2 = 0; o2 < 2; ++o2) {
                        const uint32_t dst = map_to_cta(ap_s, 2 * pg + o2) + off;
                        st_cluster_b128(dst, hi);
                        st_cluster_b128(dst + pb, lo);
                    }
                }
            }
            fence_async_proxy();
            __syncwarp();
            if (lane < kCS) arrive_remote(map_to_cta(cbar1_s, lane));     // second exchange

            // ---- 5. second projection: partial over this head / chunk, added into x_out -----------------------------
            // The residual x_in and the bias are one more term of the sum: the cluster with c == r mod n_work adds
            // them for row r, while the MMAs of the second projection run.
            const int f = quarter * 32 + lane;
            const bool f_ok = f < of;
            const int half = ww < 4 ? 0 : 1;
            const int col0 = half * (N / 2), col1 = min(col0 + N / 2, n_rows);
            if (f_ok) {
                const float bias = p.bias2 ? to_f32(p.bias2[j * of + f]) : 0.f;
                int r = col0 + ((c - col0 % n_work) + n_work) % n_work;      // first row >= col0 with r mod n_work == c
                while (r < col1) {
                    float res[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int ri4 = r + i * n_work;
                        res[i] = ri4 < col1 ? p.x_in[(size_t)ri4 * d + j * of + f] + bias : 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int ri4 = r + i * n_work;
                        if (ri4 < col1) atomicAdd(p.x_out + (size_t)ri4 * d + j * of + f, res[i]);
                    }
                    r += 4 * n_work;
                }
            }
            ok = mbar_wait(&bar_d2, 0, &abort_flag) && ok;
            tc_fence_after_sync();
            if (ok && f_ok) {
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + 2 * N;
                for (int c0 = (col0 / 16) * 16; c0 < col1; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + c0, v);
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) {
                        const int r = c0 + jj;
                        if (r >= col0 && r < col1) atomicAdd(p.x_out + (size_t)r * d + j * of + f, v[jj]);
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                              // nobody writes into a CTA that has left
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(&p.state->error, kErrTimeout);
}

}  // namespace cl
}  // namespace aed
