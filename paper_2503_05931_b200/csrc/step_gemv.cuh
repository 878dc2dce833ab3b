// Decode-step projections for steps of at most 64 rows.
//
//   out[r, o] += sum_k B(r, k) * W[o, k]      (+ bias[o] from the CTA of the first k-split)
//
// Same contract, parameters and side jobs as step_gemm.cuh (B_PLAIN / B_GAMMA / B_LN_RELU, two weight matrices per
// launch), different mechanics.  With a handful of rows a projection launch is a chain of dependent hand-overs, not
// arithmetic: in the tcgen05 form the activation rows go registers -> shared memory -> proxy fence -> barrier -> MMA
// warp -> tensor memory -> registers -> shared memory -> reductions.  Here each of 8 warps owns 16 output features
// and the rows are the N = 8 columns of warp-level MMAs (m16n8k16, bf16 x bf16 -> fp32): after the dependency wait a
// thread loads exactly the activation values of its B fragments from global memory (L2), splits them into a bf16 high
// and low part in registers, multiplies with A fragments read by ldmatrix from the weight tiles that TMA brought in
// before the wait, transposes its 16 x 8 result through 512 bytes of shared memory and issues one 16-byte reduction.
// No tensor memory, no proxy fence, no cross-warp barrier on the critical path, and 16 to 32 KB of shared memory per
// CTA, so more CTAs of this and of the next kernel are resident at once.  Every warp fetches and splits the same
// activation values, which only pays up to about 4 rows; the second kernel below shares them through shared memory.
//
// A CTA covers 128 output features x at most 2 k-blocks of 64; the host picks the k-splits accordingly and falls back
// to the tcgen05 kernel otherwise.
#pragma once
#include "step_gemm.cuh"

namespace aed {
namespace sv {

using namespace tc;
using sg::StepGemmParams;
using sg::B_PLAIN;
using sg::B_GAMMA;
using sg::B_LN_RELU;

constexpr int kSvThreads = 320;       // warps 0..7: 16 output features each; warps 8..9: weight copies and side jobs
constexpr int kSvMaxKb = 2;

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// byte offset of the 16-byte chunk `chunk` of row `row` in a 128-byte-swizzled tile of 128-byte rows
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return static_cast<uint32_t>(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// two values -> packed bf16 high parts and packed bf16 low parts (value - high)
__device__ __forceinline__ void split2(float a, float b, uint32_t &hi, uint32_t &lo)
{
    const __nv_bfloat16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
    __nv_bfloat162 h = __halves2bfloat162(ha, hb);
    hi = *reinterpret_cast<uint32_t *>(&h);
    lo = sg::pack_bf16(a - __bfloat162float(ha), b - __bfloat162float(hb));
}

// grid: x = 128-feature tiles (of both matrices), y = k-splits.  Dynamic smem: kSvMaxKb weight tiles of 16 KB + 1024.
// kNT: row tiles of 8 (this form is used with one: up to 8 rows).
template <int MODE, int kNT>
__global__ void __launch_bounds__(kSvThreads, 2)
step_gemv_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2, StepGemmParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_a[kSvMaxKb];
    __shared__ int abort_flag;
    __shared__ float red_s[2], red_q[2];
    __shared__ float s_g[kSvMaxKb * kBlockK], s_c1[kSvMaxKb * kBlockK], s_c2[kSvMaxKb * kBlockK];      // per-k constants of this CTA's k range
    __shared__ __align__(16) float s_t[8][8][16 + 4];          // per warp: 8 rows x 16 features (+ pad), for the transposition

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool second_w = p.tiles_first > 0 && static_cast<int>(blockIdx.x) >= p.tiles_first;
    const CUtensorMap *mw = second_w ? &map_w2 : &map_w;
    const int a0 = (second_w ? static_cast<int>(blockIdx.x) - p.tiles_first : static_cast<int>(blockIdx.x)) * kTileM;
    const int a_rows = second_w ? p.a_rows2 : p.a_rows;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * blockIdx.y) / gridDim.y);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (blockIdx.y + 1)) / gridDim.y);
    const int n_kb = min(kb_end - kb_begin, kSvMaxKb);          // (the host never asks for more)
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSvMaxKb; ++s) mbar_init(&bar_a[s], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    sg::pdl_launch_dependents();

    if (warp >= 8) {
        // ---- weight copies (independent of every earlier kernel), then the side jobs --------------------------
        if (warp == 8 && lane == 0) {
            prefetch_tensormap(mw);
            for (int i = 0; i < n_kb; ++i) {
                mbar_expect_tx(&bar_a[i], kATileBytes);
                tma_load_2d(tiles + static_cast<size_t>(i) * kATileBytes, mw, (kb_begin + i) * kBlockK, a0, &bar_a[i]);
            }
        }
        const int st = threadIdx.x - 256;                 // 0..63
        const int cta = blockIdx.x + gridDim.x * blockIdx.y;
        const int n_cta = gridDim.x * gridDim.y;
        sg::side_prefetch(p, cta, n_cta, st);
        sg::pdl_wait();
        sg::side_after_wait(p, cta, n_cta, st, lane, warp - 8, red_s, red_q);
        return;
    }

    // ---- compute warps -------------------------------------------------------------------------------------
    // static per-k constants of this CTA's k range into shared memory (before the dependency wait)
    const __nv_bfloat16 *const gamma = second_w ? p.gamma2 : p.gamma;
    for (int i = threadIdx.x; i < n_kb * kBlockK; i += 256) {
        const int k = kb_begin * kBlockK + i;
        if (MODE == B_GAMMA) s_g[i] = to_f32(gamma[k]);
        if (MODE == B_LN_RELU) { s_c1[i] = p.c1[k]; s_c2[i] = p.c2[k]; }
    }
    const int f_lo = a0 + warp * 16 + (lane >> 2);             // this thread's accumulator rows: features f_lo and f_lo + 8
    float bias_lo = 0.f, bias_hi = 0.f;
    if (blockIdx.y == 0) {
        if (second_w) {
            if (p.bias2) { if (f_lo < a_rows) bias_lo = p.bias2[f_lo]; if (f_lo + 8 < a_rows) bias_hi = p.bias2[f_lo + 8]; }
        } else if (p.bias) {
            if (f_lo < a_rows) bias_lo = to_f32(p.bias[f_lo]);
            if (f_lo + 8 < a_rows) bias_hi = to_f32(p.bias[f_lo + 8]);
        }
    }
    float *const out = second_w ? p.out2 : p.out;
    const int ldo = second_w ? p.ldo2 : p.ldo;
    asm volatile("bar.sync 2, 256;" ::: "memory");           // the constants are in place (still before the wait)

    sg::pdl_wait();
    const int n_rows = p.state->n_active;
    // B fragments: column n = lane / 4 is row nt * 8 + n of the step, rows k0 + {0, 1, 8, 9} with k0 = 16 ks + 2 (lane % 4)
    const int kq = (lane & 3) * 2;
    float2 xa[kNT][kSvMaxKb][4], xb[kNT][kSvMaxKb][4];
    float2 stats[kNT];
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt) {
        const int r = nt * 8 + (lane >> 2);
        const bool live = r < n_rows;
        const float *src = p.src + static_cast<size_t>(live ? r : 0) * p.ld_src + kb_begin * kBlockK + kq;
        stats[nt] = (MODE == B_LN_RELU && live) ? p.stats_in[r] : make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kSvMaxKb; ++i)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                if (live && i < n_kb) {
                    xa[nt][i][ks] = *reinterpret_cast<const float2 *>(src + i * kBlockK + ks * 16);
                    xb[nt][i][ks] = *reinterpret_cast<const float2 *>(src + i * kBlockK + ks * 16 + 8);
                } else {
                    xa[nt][i][ks] = make_float2(0.f, 0.f);
                    xb[nt][i][ks] = make_float2(0.f, 0.f);
                }
            }
    }
    float acc_h[kNT][4], acc_l[kNT][4];
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc_h[nt][j] = 0.f; acc_l[nt][j] = 0.f; }

    bool ok = true;
#pragma unroll
    for (int i = 0; i < kSvMaxKb; ++i) {
        if (i >= n_kb || !ok) break;
        ok = mbar_wait(&bar_a[i], 0, &abort_flag);
        if (!ok) break;
        const uint32_t wt = smem_u32(tiles + static_cast<size_t>(i) * kATileBytes);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(wt + swz(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), a);
            const int kl = i * kBlockK + ks * 16 + kq;           // index into the per-k constants
#pragma unroll
            for (int nt = 0; nt < kNT; ++nt) {
                float2 u = xa[nt][i][ks], v = xb[nt][i][ks];
                if (MODE == B_GAMMA) {
                    u.x *= s_g[kl]; u.y *= s_g[kl + 1]; v.x *= s_g[kl + 8]; v.y *= s_g[kl + 9];
                } else if (MODE == B_LN_RELU) {
                    const float2 st = stats[nt];
                    u.x = fmaxf(fmaf(st.y, u.x - st.x * s_c1[kl], s_c2[kl]), 0.f);
                    u.y = fmaxf(fmaf(st.y, u.y - st.x * s_c1[kl + 1], s_c2[kl + 1]), 0.f);
                    v.x = fmaxf(fmaf(st.y, v.x - st.x * s_c1[kl + 8], s_c2[kl + 8]), 0.f);
                    v.y = fmaxf(fmaf(st.y, v.y - st.x * s_c1[kl + 9], s_c2[kl + 9]), 0.f);
                    if (nt * 8 + (lane >> 2) >= n_rows) { u = make_float2(0.f, 0.f); v = u; }      // rows past the end stay zero
                }
                uint32_t h0, l0, h1, l1;
                split2(u.x, u.y, h0, l0);
                split2(v.x, v.y, h1, l1);
                mma_16816(acc_h[nt], a, h0, h1);
                mma_16816(acc_l[nt], a, l0, l1);
            }
        }
    }
    if (!ok) {
        // gave up on a weight copy: let the copies that were requested land before the block's memory goes away
        if (lane == 0 && warp == 0) {
            for (int i = 0; i < n_kb; ++i) {
                const long long start = clock64();
                while (!mbar_try_wait(&bar_a[i], 0) && clock64() - start < kWaitCycles / 8) {}
            }
            atomicExch(&p.state->error, kErrTimeout);
        }
        return;
    }
    // ---- 16 features x 8 rows per warp -> [row][feature] in shared memory -> one 16-byte reduction per lane ----------
    // accumulator element j of a thread: feature (lane / 4) + 8 (j / 2), row 2 (lane % 4) + (j % 2)
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt) {
        float (*t)[16 + 4] = s_t[warp];
        __syncwarp();
        t[kq][lane >> 2] = acc_h[nt][0] + acc_l[nt][0] + bias_lo;
        t[kq + 1][lane >> 2] = acc_h[nt][1] + acc_l[nt][1] + bias_lo;
        t[kq][(lane >> 2) + 8] = acc_h[nt][2] + acc_l[nt][2] + bias_hi;
        t[kq + 1][(lane >> 2) + 8] = acc_h[nt][3] + acc_l[nt][3] + bias_hi;
        __syncwarp();
        const int rr = lane >> 2, f4 = (lane & 3) * 4;         // row of the tile, first of 4 consecutive features
        const float4 v = *reinterpret_cast<const float4 *>(&t[rr][f4]);
        const int r = nt * 8 + rr, o = a0 + warp * 16 + f4;
        if (r < n_rows) {
            float *dst = out + static_cast<size_t>(r) * ldo + o;
            if (o + 3 < a_rows) sg::red_add_v4(dst, v);
            else {
                if (o + 0 < a_rows) atomicAdd(dst + 0, v.x);
                if (o + 1 < a_rows) atomicAdd(dst + 1, v.y);
                if (o + 2 < a_rows) atomicAdd(dst + 2, v.z);
            }
        }
    }
}

// The same projection for steps of 9 to 32 rows.  Loading B fragments straight from global memory makes every one of
// the 8 warps fetch and split the same activation values; beyond a handful of rows that traffic costs more than one
// hand-over through shared memory.  Here the 256 compute threads load the rows' k range once (coalesced 16-byte loads),
// apply the transform, write bf16 high and low planes [row][k] into shared memory (row pitch padded against bank
// conflicts), meet at one named barrier, and every warp reads its B fragments with ldmatrix.  A CTA covers at most 32
// rows: with 64 the accumulators alone take 64 registers, one CTA fits per SM and the tcgen05 kernel is faster (1350
// against 1195 us per step of the 24-layer model); launches of up to 64 rows put two row halves on grid.z.
// kKB: most k-blocks per CTA (2, or 4 for the launches of 33 to 64 rows, which halve the k-splits and put two row
// halves on grid.z instead: the same number of CTAs, half the reduction traffic).
__host__ __device__ constexpr int sv_pitch(int kb) { return kb * kBlockK * 2 + 16; }          // bytes per row of a plane: the CTA's k range in bf16 + pad
__host__ __device__ constexpr int sv_staged_smem(int nt, int kb = kSvMaxKb) { return kb * kATileBytes + 2 * nt * 8 * sv_pitch(kb) + 1024; }

// grid: x = 128-feature tiles, y = k-splits, z = row tiles of kNT * 8 rows.
template <int MODE, int kNT, int kKB = kSvMaxKb>
__global__ void __launch_bounds__(kSvThreads, 2)
step_gemv_staged_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2, StepGemmParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_a[kKB];
    __shared__ int abort_flag;
    __shared__ float red_s[2], red_q[2];
    __shared__ __align__(16) float s_g[kKB * kBlockK], s_c1[kKB * kBlockK], s_c2[kKB * kBlockK];
    __shared__ __align__(16) float s_t[8][8][16 + 4];

    static_assert(kNT == 2 || kNT == 4, "row tiles are read in pairs");
    constexpr int kRows = kNT * 8, kSvPitch = sv_pitch(kKB), kF4 = kKB * kBlockK / 4;      // kF4: 16-byte loads per row
    const int row0 = blockIdx.z * kRows;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool second_w = p.tiles_first > 0 && static_cast<int>(blockIdx.x) >= p.tiles_first;
    const CUtensorMap *mw = second_w ? &map_w2 : &map_w;
    const int a0 = (second_w ? static_cast<int>(blockIdx.x) - p.tiles_first : static_cast<int>(blockIdx.x)) * kTileM;
    const int a_rows = second_w ? p.a_rows2 : p.a_rows;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * blockIdx.y) / gridDim.y);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (blockIdx.y + 1)) / gridDim.y);
    const int n_kb = min(kb_end - kb_begin, kKB);
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *plane_hi = tiles + kKB * kATileBytes, *plane_lo = plane_hi + kRows * kSvPitch;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kKB; ++s) mbar_init(&bar_a[s], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    sg::pdl_launch_dependents();

    if (warp >= 8) {
        if (warp == 8 && lane == 0) {
            prefetch_tensormap(mw);
            for (int i = 0; i < n_kb; ++i) {
                mbar_expect_tx(&bar_a[i], kATileBytes);
                tma_load_2d(tiles + static_cast<size_t>(i) * kATileBytes, mw, (kb_begin + i) * kBlockK, a0, &bar_a[i]);
            }
        }
        const int st = threadIdx.x - 256;
        const int cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        const int n_cta = gridDim.x * gridDim.y * gridDim.z;
        sg::side_prefetch(p, cta, n_cta, st);
        sg::pdl_wait();
        sg::side_after_wait(p, cta, n_cta, st, lane, warp - 8, red_s, red_q);
        return;
    }

    const __nv_bfloat16 *const gamma = second_w ? p.gamma2 : p.gamma;
    for (int i = threadIdx.x; i < n_kb * kBlockK; i += 256) {
        const int k = kb_begin * kBlockK + i;
        if (MODE == B_GAMMA) s_g[i] = to_f32(gamma[k]);
        if (MODE == B_LN_RELU) { s_c1[i] = p.c1[k]; s_c2[i] = p.c2[k]; }
    }
    const int f_lo = a0 + warp * 16 + (lane >> 2);
    float bias_lo = 0.f, bias_hi = 0.f;
    if (blockIdx.y == 0) {
        if (second_w) {
            if (p.bias2) { if (f_lo < a_rows) bias_lo = p.bias2[f_lo]; if (f_lo + 8 < a_rows) bias_hi = p.bias2[f_lo + 8]; }
        } else if (p.bias) {
            if (f_lo < a_rows) bias_lo = to_f32(p.bias[f_lo]);
            if (f_lo + 8 < a_rows) bias_hi = to_f32(p.bias[f_lo + 8]);
        }
    }
    float *const out = second_w ? p.out2 : p.out;
    const int ldo = second_w ? p.ldo2 : p.ldo;
    asm volatile("bar.sync 2, 256;" ::: "memory");

    sg::pdl_wait();
    const int n_rows = p.state->n_active;
    // ---- the rows' k range -> planes: element e of the tile is row e / kF4, floats 4 (e % kF4) .. + 3 ------------------
    constexpr int kPer = kRows * kF4 / 256;                    // 16-byte loads per thread
    float4 xv[kPer];
    float2 st[kPer];
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const int e = threadIdx.x + 256 * j, rl = e / kF4, r = row0 + rl, c4 = e % kF4;
        const bool live = r < n_rows && c4 * 4 < n_kb * kBlockK;
        xv[j] = live ? *reinterpret_cast<const float4 *>(p.src + static_cast<size_t>(r) * p.ld_src + kb_begin * kBlockK + c4 * 4)
                     : make_float4(0.f, 0.f, 0.f, 0.f);
        st[j] = (MODE == B_LN_RELU && r < n_rows) ? p.stats_in[r] : make_float2(0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const int e = threadIdx.x + 256 * j, rl = e / kF4, r = row0 + rl, c4 = e % kF4;
        float y[4] = {xv[j].x, xv[j].y, xv[j].z, xv[j].w};
        if (MODE == B_GAMMA) {
            const float4 g = *reinterpret_cast<const float4 *>(&s_g[c4 * 4]);
            y[0] *= g.x; y[1] *= g.y; y[2] *= g.z; y[3] *= g.w;
        } else if (MODE == B_LN_RELU) {
            const float4 c1 = *reinterpret_cast<const float4 *>(&s_c1[c4 * 4]), c2 = *reinterpret_cast<const float4 *>(&s_c2[c4 * 4]);
            const float cc1[4] = {c1.x, c1.y, c1.z, c1.w}, cc2[4] = {c2.x, c2.y, c2.z, c2.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) y[q] = (r < n_rows) ? fmaxf(fmaf(st[j].y, y[q] - st[j].x * cc1[q], cc2[q]), 0.f) : 0.f;
        }
        uint32_t h0, l0, h1, l1;
        split2(y[0], y[1], h0, l0);
        split2(y[2], y[3], h1, l1);
        *reinterpret_cast<uint2 *>(plane_hi + rl * kSvPitch + c4 * 8) = make_uint2(h0, h1);
        *reinterpret_cast<uint2 *>(plane_lo + rl * kSvPitch + c4 * 8) = make_uint2(l0, l1);
    }
    asm volatile("bar.sync 2, 256;" ::: "memory");           // planes complete

    float acc_h[kNT][4], acc_l[kNT][4];
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc_h[nt][j] = 0.f; acc_l[nt][j] = 0.f; }
    bool ok = true;
    // ldmatrix addresses of the B fragments: matrices (rows 0-7, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 0-7), (rows 8-15, k 8-15)
    const uint32_t b_off = static_cast<uint32_t>(((lane & 7) + ((lane >> 4) << 3)) * kSvPitch + ((lane >> 3) & 1) * 16);
    const uint32_t hi_base = smem_u32(plane_hi), lo_base = smem_u32(plane_lo);
#pragma unroll
    for (int i = 0; i < kKB; ++i) {
        if (i >= n_kb || !ok) break;
        ok = mbar_wait(&bar_a[i], 0, &abort_flag);
        if (!ok) break;
        const uint32_t wt = smem_u32(tiles + static_cast<size_t>(i) * kATileBytes);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(wt + swz(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), a);
            const uint32_t kbyte = static_cast<uint32_t>((i * kBlockK + ks * 16) * 2);
#pragma unroll
            for (int np = 0; np < kNT; np += 2) {                // two row tiles of 8 per ldmatrix
                uint32_t bh[4], bl[4];
                ldmatrix_x4(hi_base + np * 8 * kSvPitch + b_off + kbyte, bh);
                ldmatrix_x4(lo_base + np * 8 * kSvPitch + b_off + kbyte, bl);
                mma_16816(acc_h[np], a, bh[0], bh[1]);
                mma_16816(acc_l[np], a, bl[0], bl[1]);
                mma_16816(acc_h[np + 1], a, bh[2], bh[3]);
                mma_16816(acc_l[np + 1], a, bl[2], bl[3]);
            }
        }
    }
    if (!ok) {
        if (lane == 0 && warp == 0) {
            for (int i = 0; i < n_kb; ++i) {
                const long long start = clock64();
                while (!mbar_try_wait(&bar_a[i], 0) && clock64() - start < kWaitCycles / 8) {}
            }
            atomicExch(&p.state->error, kErrTimeout);
        }
        return;
    }
    const int kq = (lane & 3) * 2;
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt) {
        float (*t)[16 + 4] = s_t[warp];
        __syncwarp();
        t[kq][lane >> 2] = acc_h[nt][0] + acc_l[nt][0] + bias_lo;
        t[kq + 1][lane >> 2] = acc_h[nt][1] + acc_l[nt][1] + bias_lo;
        t[kq][(lane >> 2) + 8] = acc_h[nt][2] + acc_l[nt][2] + bias_hi;
        t[kq + 1][(lane >> 2) + 8] = acc_h[nt][3] + acc_l[nt][3] + bias_hi;
        __syncwarp();
        const int rr = lane >> 2, f4 = (lane & 3) * 4;
        const float4 v = *reinterpret_cast<const float4 *>(&t[rr][f4]);
        const int r = row0 + nt * 8 + rr, o = a0 + warp * 16 + f4;
        if (r < n_rows) {
            float *dst = out + static_cast<size_t>(r) * ldo + o;
            if (o + 3 < a_rows) sg::red_add_v4(dst, v);
            else {
                if (o + 0 < a_rows) atomicAdd(dst + 0, v.x);
                if (o + 1 < a_rows) atomicAdd(dst + 1, v.y);
                if (o + 2 < a_rows) atomicAdd(dst + 2, v.z);
            }
        }
    }
}

}  // namespace sv
}  // namespace aed
