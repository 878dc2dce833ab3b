// Final LayerNorm + vocabulary projection + greedy argmax for steps of at most 16 rows, in one kernel.
//
//   z[r, o] = rstd_r * (sum_k (gamma[k] x[r, k]) Wout[o, k] - mean_r * c1[o]) + c2[o]
//   c1[o] = sum_k gamma[k] Wout[o, k],  c2[o] = sum_k beta[k] Wout[o, k] + b_out[o]      (built at create)
//
// which is LayerNorm(x) Wout^T + b_out with the normalisation folded as in the layer projections (step_gemm.cuh).  With
// few rows the separate normalisation kernel and the tcgen05 projection are two links of the step's dependency chain
// whose work is a few microseconds of weight streaming; here one CTA per 128 vocabulary rows
//   * streams its 128 x d weight tile through a ring of 16 KB stages from the moment it becomes resident (the weights
//     do not depend on the step; four issuing threads, since a thread's copies complete one after the other),
//   * after the dependency wait lets every warp load two rows of x, compute their (mean, rstd) in registers and write
//     gamma * x as bf16 high and low planes into shared memory,
//   * multiplies by warp-level MMAs (m16n8k16; 8 warps x 16 vocabulary rows, the step's rows as two N = 8 tiles),
//   * and finishes each row: logits for the caller if asked, and one 64-bit atomicMax per row and CTA on the packed
//     (value, lowest index) key that the step's last kernel decodes.
#pragma once
#include "step_gemv.cuh"

namespace aed {
namespace vg {

using namespace tc;

constexpr int kVgComputeWarps = 8, kVgProducers = 4;
constexpr int kVgThreads = (kVgComputeWarps + kVgProducers) * 32;
constexpr int kVgStages = 8;                       // multiple of the producers: every stage has one owner
constexpr int kVgRows = 16;

struct VocabGemvParams {
    int vocab, d_model;
    const float *x;                    // [rows, d_model] residual stream after the last layer
    const __nv_bfloat16 *gamma;        // final LayerNorm gain [d_model]
    const float *c1, *c2;              // fold constants [vocab] each
    float eps;
    float *logits_out;                 // [batch, vocab] by utterance, or nullptr
    unsigned long long *keys;          // [rows]
    const int32_t *active_list;
    DecState *state;
};

__host__ __device__ constexpr int vg_pitch(int d_model) { return d_model * 2 + 16; }       // bytes per row of a plane
__host__ __device__ constexpr int vg_smem(int d_model) { return kVgStages * kATileBytes + 2 * kVgRows * vg_pitch(d_model) + 1024; }

// grid: one CTA per 128 vocabulary rows.
__global__ void __launch_bounds__(kVgThreads, 1)
vocab_gemv_kernel(const __grid_constant__ CUtensorMap map_w, VocabGemvParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_full[kVgStages];
    __shared__ __align__(8) uint64_t bar_empty[kVgStages];
    __shared__ int abort_flag;
    __shared__ float2 s_stats[kVgRows];
    __shared__ __align__(16) float s_t[kVgComputeWarps][8][16 + 4];
    __shared__ unsigned long long s_keys[kVgComputeWarps][kVgRows];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int a0 = blockIdx.x * kTileM;
    const int k_blocks = p.d_model / kBlockK;
    const int pitch = vg_pitch(p.d_model);
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *plane_hi = tiles + kVgStages * kATileBytes, *plane_lo = plane_hi + kVgRows * pitch;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kVgStages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], kVgComputeWarps); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    sg::pdl_launch_dependents();

    if (warp >= kVgComputeWarps) {
        // ---- weight tiles: static data, streamed from the start ---------------------------------------------------
        if (lane == 0) {
            const int me = warp - kVgComputeWarps;
            prefetch_tensormap(&map_w);
            int issued = -1;
            for (int i = me; i < k_blocks; i += kVgProducers) {
                const int s = i % kVgStages;
                if (i >= kVgStages && !mbar_wait(&bar_empty[s], ((i / kVgStages) - 1) & 1, &abort_flag)) break;
                mbar_expect_tx(&bar_full[s], kATileBytes);
                tma_load_2d(tiles + static_cast<size_t>(s) * kATileBytes, &map_w, i * kBlockK, a0, &bar_full[s]);
                issued = i;
            }
            if (abort_flag && issued >= 0) {
                const long long start = clock64();
                while (!mbar_try_wait(&bar_full[issued % kVgStages], (issued / kVgStages) & 1) && clock64() - start < kWaitCycles / 8) {}
            }
        }
        return;
    }

    // ---- rows 2 * warp and 2 * warp + 1: statistics and planes ------------------------------------------------------
    sg::pdl_wait();
    const int n_rows = p.state->n_active;
    const int per_lane = p.d_model / 128;                     // 16-byte loads per lane and row (d_model is a multiple of 128 here)
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const int r = 2 * warp + rr;
        if (r < n_rows) {
            const float *xr = p.x + static_cast<size_t>(r) * p.d_model;
            float s = 0.f;
            for (int i = 0; i < per_lane; ++i) {
                const float4 v = *reinterpret_cast<const float4 *>(xr + (lane + 32 * i) * 4);
                s += (v.x + v.y) + (v.z + v.w);
            }
            const float mean = warp_sum(s) / p.d_model;
            float q = 0.f;
            for (int i = 0; i < per_lane; ++i) {
                const int k = (lane + 32 * i) * 4;
                const float4 v = *reinterpret_cast<const float4 *>(xr + k);      // second read: from L1
                const float d0 = v.x - mean, d1 = v.y - mean, d2 = v.z - mean, d3 = v.w - mean;
                q += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
                float g[4];
                load4(p.gamma + k, g);
                uint32_t h0, l0, h1, l1;
                sv::split2(v.x * g[0], v.y * g[1], h0, l0);
                sv::split2(v.z * g[2], v.w * g[3], h1, l1);
                *reinterpret_cast<uint2 *>(plane_hi + r * pitch + k * 2) = make_uint2(h0, h1);
                *reinterpret_cast<uint2 *>(plane_lo + r * pitch + k * 2) = make_uint2(l0, l1);
            }
            q = warp_sum(q);
            if (lane == 0) s_stats[r] = make_float2(mean, rsqrtf(q / p.d_model + p.eps));
        } else {
            for (int i = 0; i < per_lane; ++i) {
                const int k = (lane + 32 * i) * 4;
                *reinterpret_cast<uint2 *>(plane_hi + r * pitch + k * 2) = make_uint2(0u, 0u);
                *reinterpret_cast<uint2 *>(plane_lo + r * pitch + k * 2) = make_uint2(0u, 0u);
            }
            if (lane == 0) s_stats[r] = make_float2(0.f, 0.f);
        }
    }
    asm volatile("bar.sync 2, 256;" ::: "memory");           // planes and statistics complete

    // ---- 16 vocabulary rows per warp x 16 step rows ------------------------------------------------------------------
    float acc_h[2][4], acc_l[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc_h[nt][j] = 0.f; acc_l[nt][j] = 0.f; }
    const uint32_t b_off = static_cast<uint32_t>(((lane & 7) + ((lane >> 4) << 3)) * pitch + ((lane >> 3) & 1) * 16);
    const uint32_t hi_base = smem_u32(plane_hi), lo_base = smem_u32(plane_lo);
    bool ok = true;
    for (int i = 0; i < k_blocks; ++i) {
        const int s = i % kVgStages;
        ok = mbar_wait(&bar_full[s], (i / kVgStages) & 1, &abort_flag);
        if (!ok) break;
        const uint32_t wt = smem_u32(tiles + static_cast<size_t>(s) * kATileBytes);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t a[4], bh[4], bl[4];
            sv::ldmatrix_x4(wt + sv::swz(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), a);
            const uint32_t kbyte = static_cast<uint32_t>((i * kBlockK + ks * 16) * 2);
            sv::ldmatrix_x4(hi_base + b_off + kbyte, bh);
            sv::ldmatrix_x4(lo_base + b_off + kbyte, bl);
            sv::mma_16816(acc_h[0], a, bh[0], bh[1]);
            sv::mma_16816(acc_l[0], a, bl[0], bl[1]);
            sv::mma_16816(acc_h[1], a, bh[2], bh[3]);
            sv::mma_16816(acc_l[1], a, bl[2], bl[3]);
        }
        __syncwarp();                                           // every lane has read the stage
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_empty[s])) : "memory");
    }
    if (!ok) {
        if (threadIdx.x == 0) atomicExch(&p.state->error, kErrTimeout);
        return;
    }
    // ---- per row: fold, logits, argmax key ----------------------------------------------------------------------------
    const int kq = (lane & 3) * 2;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        float (*t)[16 + 4] = s_t[warp];
        __syncwarp();
        t[kq][lane >> 2] = acc_h[nt][0] + acc_l[nt][0];
        t[kq + 1][lane >> 2] = acc_h[nt][1] + acc_l[nt][1];
        t[kq][(lane >> 2) + 8] = acc_h[nt][2] + acc_l[nt][2];
        t[kq + 1][(lane >> 2) + 8] = acc_h[nt][3] + acc_l[nt][3];
        __syncwarp();
        const int rr = lane >> 2, f4 = (lane & 3) * 4;         // row of the tile, first of 4 consecutive vocabulary rows
        const float4 raw = *reinterpret_cast<const float4 *>(&t[rr][f4]);
        const int r = nt * 8 + rr, o = a0 + warp * 16 + f4;
        const float2 st = s_stats[r];
        const float rawv[4] = {raw.x, raw.y, raw.z, raw.w};
        float z[4];
        unsigned long long key = 0ull;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool o_ok = o + j < p.vocab;
            z[j] = o_ok ? fmaf(st.y, rawv[j] - st.x * p.c1[o + j], p.c2[o + j]) : 0.f;
            if (o_ok && r < n_rows) {
                const unsigned long long kj = argmax_key(z[j], static_cast<uint32_t>(o + j));
                key = kj > key ? kj : key;
            }
        }
        if (r < n_rows && p.logits_out) {
            float *dst = p.logits_out + static_cast<size_t>(p.active_list[r]) * p.vocab + o;
            if (o + 3 < p.vocab && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) *reinterpret_cast<float4 *>(dst) = make_float4(z[0], z[1], z[2], z[3]);
            else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (o + j < p.vocab) dst[j] = z[j];
            }
        }
        // the 4 lanes that share a row, then this warp's entry for the row
        unsigned long long other = __shfl_xor_sync(0xffffffffu, key, 1);
        key = other > key ? other : key;
        other = __shfl_xor_sync(0xffffffffu, key, 2);
        key = other > key ? other : key;
        if ((lane & 3) == 0) s_keys[warp][r] = key;
    }
    asm volatile("bar.sync 2, 256;" ::: "memory");
    if (threadIdx.x < kVgRows && static_cast<int>(threadIdx.x) < n_rows) {
        unsigned long long key = 0ull;
#pragma unroll
        for (int w = 0; w < kVgComputeWarps; ++w) key = s_keys[w][threadIdx.x] > key ? s_keys[w][threadIdx.x] : key;
        if (key != 0ull) atomicMax(p.keys + threadIdx.x, key);
    }
}

}  // namespace vg
}  // namespace aed
