// Decode-step projection on tensor cores with the activation operand built in the kernel.
//
//   out[r, o] += sum_k B(r, k) * W[o, k]      (+ bias[o] from the CTA of the first k-split)
//
// W tiles (128 output features x 64 k, bf16) arrive by TMA; they do not depend on earlier kernels, so they are
// requested before the programmatic-dependency wait and stream in while the previous kernel drains.
// The activation tile B is produced by four warps straight from fp32 sources into the 128-byte-swizzled layout the
// MMA reads, as a bf16 high plane and a bf16 low plane (value - high), with one of three transforms fused:
//   B_PLAIN    B = src                                   (attention output -> output projection)
//   B_GAMMA    B = gamma[k] * src                        (LayerNorm folded into the projection, see below)
//   B_LN_RELU  B = relu(rstd_r * (src - mean_r * c1[k]) + c2[k])   (FFN hidden layer from the folded first GEMM)
//   B_PLANES   B arrives ready-made: bf16 high and low planes in global memory, fetched by TMA.  Steps with many rows
//              take this form: there every feature tile would otherwise convert the same activation rows again, and
//              the conversion, not the tensor cores, would set the pace.
//
// LayerNorm folding: LN(x) W^T = rstd * ((gamma*x) W^T - mean * c1) + c2 with c1[o] = sum_k gamma_k W[o,k] and
// c2[o] = sum_k beta_k W[o,k] + b[o].  The GEMM therefore runs on gamma*x without knowing the row statistics;
// whoever consumes its output applies (mean, rstd).  The statistics themselves are a side job: while the MMAs
// run, the producer warps of this kernel compute mean and rstd of the rows assigned to their CTA and store
// them for the consumer.  A second side job clears the fp32 rows a later split-K projection accumulates into.
//
// Two matrices in one launch (not in B_PLANES mode): feature tiles blockIdx.x >= tiles_first belong to a second weight
// matrix over the same activation rows, with its own tensor map (passed in the place of the low plane's), gamma,
// bias and output buffer.  This is how one launch serves two projections that depend on the same earlier kernel.
//
// A CTA walks its k-blocks through a ring of up to 4 stages (weight tile, two planes, fp32 source tile each); with
// few k-blocks per CTA (small batches, many k-splits) everything is resident at once.  Waits are bounded.
#pragma once
#include "tc_gemm.cuh"

namespace aed {
namespace sg {

using namespace tc;

constexpr int kMaxKb = 4;             // ring stages per CTA
constexpr int kSgThreads = 384;       // warp 0 TMA, warp 1 MMA, warps 2..9 activation tiles and epilogue, warps 10..11 side jobs

enum BMode { B_PLAIN = 0, B_GAMMA = 1, B_LN_RELU = 2, B_PLANES = 3 };

struct StepGemmParams {
    int a_rows;                // output features M
    int k_blocks;              // K / 64
    int n_tile;                // MMA N: rows per CTA tile (16..256, multiple of 16)
    int stages;                // ring depth, 1..kMaxKb
    int src_rows;              // rows of the source buffer (reads of rows past it are clamped)
    // activation source [rows, ld_src] fp32
    const float *src;
    int ld_src;
    const __nv_bfloat16 *gamma;    // B_GAMMA: [K]
    const float *c1, *c2;          // B_LN_RELU: [K] each
    const float2 *stats_in;        // B_LN_RELU: (mean, rstd) per row
    // epilogue
    float *out;
    int ldo;
    const __nv_bfloat16 *bias;     // added by k-split 0, may be null
    // second matrix (feature tiles tiles_first .. gridDim.x - 1); tiles_first == 0: none
    int tiles_first;
    int a_rows2;
    const __nv_bfloat16 *gamma2;   // B_GAMMA
    float *out2;
    int ldo2;
    const float *bias2;            // fp32, added by k-split 0, may be null
    // side job 1: (mean, rstd) of the rows of stats_src [rows, stats_d]
    const float *stats_src;
    float2 *stats_out;
    int stats_d;
    float eps;
    // side job 2: clear zero_buf [rows, zero_cols]
    float *zero_buf;
    int zero_cols;
    // side job 3: pull a byte range that a later kernel streams (next layer's weights) into L2
    const void *prefetch_ptr, *prefetch2_ptr;      // (the second range: the output matrix, from the last layer)
    size_t prefetch_bytes, prefetch2_bytes;
    DecState *state;
};

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&p);
}

// 8 values -> one 16-byte chunk of the high plane and one of the low plane
__device__ __forceinline__ void split_planes(const float (&y)[8], uint4 &hi, uint4 &lo)
{
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(y[2 * i]), h1 = __float2bfloat16_rn(y[2 * i + 1]);
        __nv_bfloat162 hp = __halves2bfloat162(h0, h1);
        h[i] = *reinterpret_cast<uint32_t *>(&hp);
        l[i] = pack_bf16(y[2 * i] - __bfloat162float(h0), y[2 * i + 1] - __bfloat162float(h1));
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// 4 floats added to 4 consecutive addresses with one reduction (16-byte aligned)
__device__ __forceinline__ void red_add_v4(float *addr, float4 v)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// ---- side jobs of a projection launch, run by 64 threads (two warps) of every CTA, off the critical path -----------
// st: 0..63 among those threads; cta / n_cta: this CTA among all CTAs of the launch.
// Static data (a later kernel's weights) into L2: no need to wait for the previous kernel.  4 KB pieces.
__device__ __forceinline__ void side_prefetch(const StepGemmParams &p, int cta, int n_cta, int st)
{
    for (int range = 0; range < 2; ++range) {
        const char *base = static_cast<const char *>(range ? p.prefetch2_ptr : p.prefetch_ptr);
        if (!base) continue;
        const size_t pieces = (range ? p.prefetch2_bytes : p.prefetch_bytes) / 4096;
        for (size_t i = static_cast<size_t>(cta) * 64 + st; i < pieces; i += static_cast<size_t>(n_cta) * 64)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(base + i * 4096), "r"(4096) : "memory");
    }
}
// After the dependency wait: clear the rows a later split-K projection accumulates into, and (mean, rstd) of the rows
// assigned to this CTA.  w: 0 or 1, which of the two warps; red_s, red_q: two floats of shared memory each.
__device__ __forceinline__ void side_after_wait(const StepGemmParams &p, int cta, int n_cta, int st, int lane, int w,
                                                float *red_s, float *red_q)
{
    const int n_rows = p.state->n_active;
    if (p.zero_buf) {
        const size_t total4 = static_cast<size_t>(n_rows) * p.zero_cols / 4;
        float4 *z = reinterpret_cast<float4 *>(p.zero_buf);
        for (size_t idx = static_cast<size_t>(cta) * 64 + st; idx < total4; idx += static_cast<size_t>(n_cta) * 64)
            z[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (p.stats_src) {
        for (int r = cta; r < n_rows; r += n_cta) {    // uniform over the two warps
            const float *xr = p.stats_src + static_cast<size_t>(r) * p.stats_d;
            float s = 0.f;
            for (int idx = st * 4; idx < p.stats_d; idx += 256) {
                const float4 v = *reinterpret_cast<const float4 *>(xr + idx);
                s += (v.x + v.y) + (v.z + v.w);
            }
            s = warp_sum(s);
            if (lane == 0) red_s[w] = s;
            asm volatile("bar.sync 1, 64;" ::: "memory");
            const float mean = (red_s[0] + red_s[1]) / p.stats_d;
            float q = 0.f;
            for (int idx = st * 4; idx < p.stats_d; idx += 256) {
                const float4 v = *reinterpret_cast<const float4 *>(xr + idx);
                const float d0 = v.x - mean, d1 = v.y - mean, d2 = v.z - mean, d3 = v.w - mean;
                q += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
            }
            q = warp_sum(q);
            if (lane == 0) red_q[w] = q;
            asm volatile("bar.sync 1, 64;" ::: "memory");
            if (st == 0) p.stats_out[r] = make_float2(mean, rsqrtf((red_q[0] + red_q[1]) / p.stats_d + p.eps));
            asm volatile("bar.sync 1, 64;" ::: "memory");
        }
    }
}

// grid: x = 128-feature tiles, y = k-splits, z = row tiles.
// Dynamic smem per k-block: weight tile 16 KB | high plane | low plane (n_tile x 128 B each) | fp32 source tile
// (n_tile x 256 B, filled by TMA, later reused to transpose the accumulator); plus 1024 for alignment.
template <int MODE>
__global__ void __launch_bounds__(kSgThreads, 2)
step_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_src,
                 const __grid_constant__ CUtensorMap map_lo, StepGemmParams p)
{
    // map_src: fp32 source tiles (B_PLAIN, B_GAMMA, B_LN_RELU) or the high plane (B_PLANES); map_lo: the low plane.
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_a[kMaxKb];
    __shared__ __align__(8) uint64_t bar_s[kMaxKb];
    __shared__ __align__(8) uint64_t bar_b[kMaxKb];
    __shared__ __align__(8) uint64_t bar_e[kMaxKb];
    __shared__ __align__(8) uint64_t bar_done;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float red_s[2], red_q[2];

    // timeline of the first producer thread of block 0 (debug builds)
    AED_TRACE_RESERVE(tcur, p.state, (threadIdx.x == 64 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) ? 10u : 0u);
    AED_TRACE_PUT_NS(p.state, tcur, 19);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool second_w = MODE != B_PLANES && p.tiles_first > 0 && static_cast<int>(blockIdx.x) >= p.tiles_first;
    const CUtensorMap *mw = second_w ? &map_lo : &map_w;
    const int a0 = (second_w ? static_cast<int>(blockIdx.x) - p.tiles_first : static_cast<int>(blockIdx.x)) * kTileM;
    const int a_rows = second_w ? p.a_rows2 : p.a_rows;
    const int row0 = blockIdx.z * p.n_tile;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * blockIdx.y) / gridDim.y);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (blockIdx.y + 1)) / gridDim.y);
    const int n_kb = kb_end - kb_begin;
    const int S = p.stages;
    // Small tiles (at most 32 rows, one or two k-blocks): the producer threads read their 8 source values per k-block
    // straight from global memory right after the dependency wait instead of waiting for a TMA copy into shared memory.
    const bool direct = MODE != B_PLANES && p.n_tile <= 32 && n_kb <= 2;

    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const int plane_bytes = p.n_tile * kBlockK * 2;
    const int src_bytes = MODE == B_PLANES ? 0 : p.n_tile * kBlockK * 4;
    const int stage_bytes = kATileBytes + 2 * plane_bytes + src_bytes;
    uint32_t tmem_cols = 32;
    while (tmem_cols < static_cast<uint32_t>(p.n_tile)) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxKb; ++s) { mbar_init(&bar_a[s], 1); mbar_init(&bar_s[s], 1); mbar_init(&bar_b[s], 8); mbar_init(&bar_e[s], 1); }
        mbar_init(&bar_done, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_slot, tmem_cols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    pdl_launch_dependents();
    AED_TRACE_PUT(p.state, tcur, 40);      // set-up done

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(mw);
            prefetch_tensormap(&map_src);
            const int pre = n_kb < S ? n_kb : S;
            for (int i = 0; i < pre; ++i) {       // weights: independent of every earlier kernel
                mbar_expect_tx(&bar_a[i], kATileBytes);
                tma_load_2d(tiles + static_cast<size_t>(i) * stage_bytes, mw, (kb_begin + i) * kBlockK, a0, &bar_a[i]);
            }
        }
        pdl_wait();
        if (lane == 0) {
            for (int i = 0; i < n_kb; ++i) {
                const int s = i % S;
                uint8_t *stage = tiles + static_cast<size_t>(s) * stage_bytes;
                if (i >= S) {                     // the stage is free once the MMAs of k-block i - S have read it
                    if (!mbar_wait(&bar_e[s], ((i / S) - 1) & 1, &abort_flag)) break;
                    mbar_expect_tx(&bar_a[s], kATileBytes);
                    tma_load_2d(stage, mw, (kb_begin + i) * kBlockK, a0, &bar_a[s]);
                }
                // fp32 activation source, written by the previous kernels
                if (MODE != B_PLANES && !direct) {
                    mbar_expect_tx(&bar_s[s], src_bytes);
                    tma_load_2d(stage + kATileBytes + 2 * plane_bytes, &map_src, (kb_begin + i) * kBlockK, row0, &bar_s[s]);
                }
            }
        }
    } else if (warp == 1) {
        pdl_wait();
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(p.n_tile);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % S;
                const uint32_t par = (i / S) & 1;
                ok = mbar_wait(MODE == B_PLANES ? &bar_s[s] : &bar_b[s], par, &abort_flag) && mbar_wait(&bar_a[s], par, &abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sa = smem_u32(tiles + static_cast<size_t>(s) * stage_bytes);
                const uint64_t da = smem_desc_sw128(sa), dh = smem_desc_sw128(sa + kATileBytes),
                               dl = smem_desc_sw128(sa + kATileBytes + plane_bytes);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(tmem_base, da + 2 * k, dh + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) mma_bf16(tmem_base, da + 2 * k, dl + 2 * k, idesc, 1u);
                if (i + S < n_kb) mma_commit(&bar_e[s]);      // someone is waiting to refill this stage
            }
            if (ok) mma_commit(&bar_done);
            else {
                // weight copies that were requested must land before the block retires
                for (int s = 0; s < S && s < n_kb; ++s) {
                    const long long start = clock64();
                    while (!mbar_try_wait(&bar_a[s], 0) && clock64() - start < kWaitCycles / 8) {}
                }
            }
        }
    } else if (warp >= 10) {
        // ---- side jobs, off the critical path --------------------------------------------------------------
        const int st = threadIdx.x - 320;                 // 0..63
        const int cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        const int n_cta = gridDim.x * gridDim.y * gridDim.z;
        side_prefetch(p, cta, n_cta, st);
        pdl_wait();
        if (MODE == B_PLANES) {
            // the activation planes of every k-block, by the first lane of these two warps (a thread's copies complete
            // one after the other); each ring stage is refilled by one of them only
            if (lane == 0) {
                const int loaders = (S % 2 == 0) ? 2 : 1, me = warp - 10;
                if (me < loaders) {
                    for (int i = me; i < n_kb; i += loaders) {
                        const int s = i % S;
                        if (i >= S && !mbar_wait(&bar_e[s], ((i / S) - 1) & 1, &abort_flag)) break;
                        uint8_t *stage = tiles + static_cast<size_t>(s) * stage_bytes;
                        mbar_expect_tx(&bar_s[s], 2 * plane_bytes);
                        tma_load_2d(stage + kATileBytes, &map_src, (kb_begin + i) * kBlockK, row0, &bar_s[s]);
                        tma_load_2d(stage + kATileBytes + plane_bytes, &map_lo, (kb_begin + i) * kBlockK, row0, &bar_s[s]);
                    }
                }
            }
        }
        side_after_wait(p, cta, n_cta, st, lane, warp - 10, red_s, red_q);
    } else {
        pdl_wait();
        AED_TRACE_PUT(p.state, tcur, 41);  // dependency resolved
        const int pt = threadIdx.x - 64;                  // 0..255 among the producer threads
        const int n_rows = p.state->n_active;
        // ---- activation tiles --------------------------------------------------------------------------
        // Thread pt owns the 16-byte output chunk c = pt & 7 (8 consecutive k) of rows (pt >> 3) + 32 j.  The fp32
        // source tile of each k-block is already on its way into shared memory (TMA, no swizzle, 256 B per row).
        // Each k-block has its own barrier, so the MMAs of one k-block run while the next is converted.
        const int c = pt & 7, rbase = pt >> 3;
        const int quarter = warp & 3;
        const int a_idx = a0 + quarter * 32 + lane;
        const bool a_ok = a_idx < a_rows;
        float bias = 0.f;
        if (blockIdx.y == 0 && a_ok) {
            if (second_w) bias = p.bias2 ? p.bias2[a_idx] : 0.f;
            else bias = p.bias ? to_f32(p.bias[a_idx]) : 0.f;
        }
        float *const out = second_w ? p.out2 : p.out;
        const int ldo = second_w ? p.ldo2 : p.ldo;
        const __nv_bfloat16 *const gamma = second_w ? p.gamma2 : p.gamma;
        float dv[2][8];
        if (direct && rbase < p.n_tile) {          // one row per thread (n_tile <= 32), both k-blocks requested at once
            const int rs = min(row0 + rbase, p.src_rows - 1);
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (i < n_kb) load8(p.src + static_cast<size_t>(rs) * p.ld_src + (kb_begin + i) * kBlockK + c * 8, dv[i]);
        }
        bool ok = true;
        for (int i = 0; MODE != B_PLANES && i < n_kb && ok; ++i) {
            const int s = i % S;
            uint8_t *stage = tiles + static_cast<size_t>(s) * stage_bytes;
            uint8_t *hi_tile = stage + kATileBytes, *lo_tile = hi_tile + plane_bytes;
            const float *src_tile = reinterpret_cast<const float *>(lo_tile + plane_bytes);
            const int k = (kb_begin + i) * kBlockK + c * 8;
            float g[8], c1[8], c2[8];
            if (MODE == B_GAMMA) load8(gamma + k, g);
            if (MODE == B_LN_RELU) { load8(p.c1 + k, c1); load8(p.c2 + k, c2); }
            if (!direct) ok = mbar_wait(&bar_s[s], (i / S) & 1, &abort_flag);
            if (!ok) break;
            for (int rl = rbase; rl < p.n_tile; rl += 32) {
                const int r = row0 + rl;
                float y[8];
                if (r < n_rows) {
                    if (direct) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] = i == 0 ? dv[0][e] : dv[1][e];
                    } else load8(src_tile + rl * kBlockK + c * 8, y);
                    if (MODE == B_GAMMA) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] *= g[e];
                    } else if (MODE == B_LN_RELU) {
                        const float2 st = p.stats_in[r];
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] = fmaxf(fmaf(st.y, y[e] - st.x * c1[e], c2[e]), 0.f);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) y[e] = 0.f;
                }
                uint4 hi, lo;
                split_planes(y, hi, lo);
                const int off = rl * 128 + ((c ^ (rl & 7)) << 4);
                *reinterpret_cast<uint4 *>(hi_tile + off) = hi;
                *reinterpret_cast<uint4 *>(lo_tile + off) = lo;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_b[s])) : "memory");
        }
        AED_TRACE_PUT(p.state, tcur, 42);  // activation tiles written
        {
        // ---- epilogue: accumulator -> shared memory (transposed) -> 16-byte reductions ---------------------------
        // Warps w and w + 4 reach the same accumulator lanes (lane quarter = warp & 3): they split the rows in 16s.
        ok = ok && mbar_wait(&bar_done, 0, &abort_flag);
        tc_fence_after_sync();
        AED_TRACE_PUT(p.state, tcur, 44);  // accumulator complete
        // every MMA has completed, so the whole stage area is free: T[r][o], 132 floats per row (bank spread)
        float *trans = reinterpret_cast<float *>(tiles);
        constexpr int kPitch = kTileM + 4;
        const int rows_here = min(p.n_tile, max(n_rows - row0, 0));
        const int second = warp >= 6 ? 1 : 0;
        // (B_PLANES: the launch reserves at least the transposition buffer, whatever the ring needs)
        const bool fits = MODE == B_PLANES || static_cast<size_t>(p.n_tile) * kPitch * 4 <= static_cast<size_t>(n_kb < S ? n_kb : S) * stage_bytes;
        if (ok && fits) {
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            for (int c0 = 16 * second; c0 < rows_here; c0 += 32) {
                float v[16];
                tmem_ld16(taddr + c0, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) trans[(c0 + j) * kPitch + quarter * 32 + lane] = v[j] + bias;
            }
        }
        AED_TRACE_PUT(p.state, tcur, 46);  // accumulator in shared memory
        asm volatile("bar.sync 2, 256;" ::: "memory");
        AED_TRACE_PUT(p.state, tcur, 47);  // all epilogue warps there
        if (ok && fits) {
            const int o4 = (pt & 31) * 4;
            for (int rl = pt >> 5; rl < rows_here; rl += 8) {
                const float4 v = *reinterpret_cast<const float4 *>(trans + rl * kPitch + o4);
                float *dst = out + static_cast<size_t>(row0 + rl) * ldo + a0 + o4;
                if (a0 + o4 + 3 < a_rows) red_add_v4(dst, v);
                else {
                    if (a0 + o4 + 0 < a_rows) atomicAdd(dst + 0, v.x);
                    if (a0 + o4 + 1 < a_rows) atomicAdd(dst + 1, v.y);
                    if (a0 + o4 + 2 < a_rows) atomicAdd(dst + 2, v.z);
                }
            }
        } else if (ok) {
            // transposition buffer too small for this shape: scalar reductions straight from the accumulator
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            for (int c0 = 16 * second; c0 < rows_here; c0 += 32) {
                float v[16];
                tmem_ld16(taddr + c0, v);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (a_ok && c0 + j < rows_here) atomicAdd(out + static_cast<size_t>(row0 + c0 + j) * ldo + a_idx, v[j] + bias);
            }
        }
        }
    }
    AED_TRACE_PUT_NS(p.state, tcur, 45);   // epilogue issued
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(&p.state->error, kErrTimeout);
}

// c1[o] = sum_k gamma[k] W[o,k];  c2[o] = sum_k beta[k] W[o,k] + bias[o]   (one warp per output feature)
__global__ void ln_fold_constants_kernel(const __nv_bfloat16 *__restrict__ w, const __nv_bfloat16 *__restrict__ gamma,
                                         const __nv_bfloat16 *__restrict__ beta, const __nv_bfloat16 *__restrict__ bias,
                                         int m, int k, float *__restrict__ c1, float *__restrict__ c2)
{
    const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (o >= m) return;
    float s1 = 0.f, s2 = 0.f;
    for (int i = lane; i < k; i += 32) {
        const float wv = to_f32(w[static_cast<size_t>(o) * k + i]);
        s1 = fmaf(to_f32(gamma[i]), wv, s1);
        s2 = fmaf(to_f32(beta[i]), wv, s2);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    if (lane == 0) { c1[o] = s1; c2[o] = s2 + (bias ? to_f32(bias[o]) : 0.f); }
}

// Two projections that meet without a nonlinearity between them, composed once at set-up:
//   C[o][i] = sum_k A[o][k] g[k] B[k][i]   (bf16, row-major [n, n]);   cb[o] = sum_k A[o][k] g[k] b[k]
// so that (g * (x + y B^T + b)) A^T = (g * x) A^T + y C^T + cb: the second projection no longer has to wait for the
// sum over all features of the first.  16 x 16 outputs per block, fp32 accumulation.
__global__ void compose_weights_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *__restrict__ g,
                                       const __nv_bfloat16 *__restrict__ b, int n, __nv_bfloat16 *__restrict__ c)
{
    __shared__ float sa[16][17], sb[16][17];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int o = blockIdx.y * 16 + ty, i = blockIdx.x * 16 + tx;
    float acc = 0.f;
    for (int k0 = 0; k0 < n; k0 += 16) {
        const int ka = k0 + tx, kb = k0 + ty;
        sa[ty][tx] = (o < n && ka < n) ? to_f32(a[static_cast<size_t>(o) * n + ka]) * to_f32(g[ka]) : 0.f;
        sb[ty][tx] = (kb < n && i < n) ? to_f32(b[static_cast<size_t>(kb) * n + i]) : 0.f;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) acc = fmaf(sa[ty][k], sb[k][tx], acc);
        __syncthreads();
    }
    if (o < n && i < n) c[static_cast<size_t>(o) * n + i] = __float2bfloat16_rn(acc);
}

__global__ void compose_bias_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *__restrict__ g,
                                    const __nv_bfloat16 *__restrict__ b, int n, float *__restrict__ cb)
{
    const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (o >= n) return;
    float s = 0.f;
    if (b)
        for (int k = lane; k < n; k += 32) s = fmaf(to_f32(a[static_cast<size_t>(o) * n + k]) * to_f32(g[k]), to_f32(b[k]), s);
    s = warp_sum(s);
    if (lane == 0) cb[o] = s;
}

}  // namespace sg
}  // namespace aed
