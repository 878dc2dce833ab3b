// Flash-decoding attention for steps with many rows (bf16 caches): the K/V-bound regime.
//
// A (row, head) pair reads one contiguous run of keys and one of values (len x 128 bytes each).  With hundreds of
// rows those runs are nearly all of a step's bytes, so the kernel is built to keep every SM streaming:
//   * persistent blocks, one per SM; block b takes the work items b, b + gridDim.x, ... of the list
//     (row-major over the compact rows, which are sorted by decreasing encoder length, so every block gets the same
//     mix of long and short runs);
//   * four producer threads pull the runs through a ring of 32 KB stages (up to 128 positions: 16 KB of keys,
//     16 KB of values) with plain bulk copies; a thread's copies complete one after the other, hence four of them,
//     each owning every fourth stage.  Cross-attention K/V is static, so the copies start before the dependency wait;
//   * one warp prepares the queries of the coming items, four at a time (LayerNorm fold, scaling, and for
//     self-attention the key and value of the position this step appends, which it also stores to the cache);
//   * sixteen consumer warps take 8 positions each of a stage, keep an online softmax per item, and hand their
//     partial (max, sum, accumulator) to a merge warp that combines them and writes the output row while the consumers
//     are already on the next item.
// Every hand-over inside the block is an mbarrier with a bounded wait.
#pragma once
#include "tc_gemm.cuh"
#include "step_kernels.cuh"

namespace aed {
namespace as {

using namespace tc;

constexpr int kStagePos = 128;                          // positions per ring stage
constexpr int kStageBytes = 2 * kStagePos * 128;        // keys then values
constexpr int kStages = 4;
constexpr int kProducers = 4;
constexpr int kConsumers = 16;                         // few warps cannot hide the latency of their own instructions
constexpr int kPosPerWarp = kStagePos / kConsumers;    // positions of a stage one consumer warp takes
constexpr int kPosIters = kPosPerWarp / 4;             // four position groups per warp
constexpr int kQSlots = 4;                              // items whose query may be prepared ahead
constexpr int kMergeSlots = 2;
constexpr int kAsThreads = (kProducers + 2 + kConsumers) * 32;     // + query warp + merge warp

struct StageMeta { int q_slot, n_pos, first, last; };  // written by the producer with the stage

struct AttnStreamParams {
    const DecState *state;
    const int4 *row_info;               // (utterance, t_u, encoder length, encoder offset) per compact row
    const float *q; int ldq;            // query rows (self: [q | k | v] rows)
    __nv_bfloat16 *cache;               // layer's self cache [batch][2][H][cap][64] or cross store [2][H][cap][64]
    int n_heads, seq_capacity;
    float scale;
    float *out; int ldo;                // [rows, d] fp32
    const float2 *ln_stats;             // per row (mean, rstd) of the LayerNorm folded into the projection
    const float *ln_c1, *ln_c2;         // fold constants per projection column
    DecState *err_state;
};

__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// grid: persistent blocks.  Dynamic shared memory: kStages * kStageBytes + 1024.
template <bool kCross>
__global__ void __launch_bounds__(kAsThreads, 1) attn_stream_kernel(const AttnStreamParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages];
    __shared__ __align__(8) uint64_t bar_q_full[kQSlots], bar_q_empty[kQSlots];
    __shared__ __align__(8) uint64_t bar_m_full[kMergeSlots], bar_m_empty[kMergeSlots];
    __shared__ StageMeta meta[kStages];
    __shared__ __align__(16) float q_s[kQSlots][kHeadDim];              // scaled queries
    __shared__ __align__(16) float new_k[kQSlots][kHeadDim], new_v[kQSlots][kHeadDim];   // self: appended position (bf16-rounded)
    __shared__ float mg_m[kMergeSlots][kConsumers], mg_l[kMergeSlots][kConsumers];
    __shared__ float mg_acc[kMergeSlots][kConsumers][kHeadDim];
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const int H = p.n_heads;
    const int n_rows = p.state->n_active;            // fixed by the step's first kernel, which completed before this launch
    const int n_items = n_rows * H;
    const int G = gridDim.x, b = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], kConsumers); }
        for (int s = 0; s < kQSlots; ++s) { mbar_init(&bar_q_full[s], 1); mbar_init(&bar_q_empty[s], kConsumers); }
        for (int s = 0; s < kMergeSlots; ++s) { mbar_init(&bar_m_full[s], kConsumers); mbar_init(&bar_m_empty[s], 1); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // length and base addresses of an item
    auto item_len = [&](const int4 &ri) { return kCross ? ri.z : ri.y; };        // static positions (self: without the new one)
    auto k_base = [&](const int4 &ri, int h) -> const __nv_bfloat16 * {
        return kCross ? p.cache + (static_cast<size_t>(0 * H + h) * p.seq_capacity + ri.w) * kHeadDim
                      : p.cache + ((static_cast<size_t>(ri.x) * 2 + 0) * H + h) * static_cast<size_t>(p.seq_capacity) * kHeadDim;
    };
    auto v_base = [&](const int4 &ri, int h) -> const __nv_bfloat16 * {
        return kCross ? p.cache + (static_cast<size_t>(1 * H + h) * p.seq_capacity + ri.w) * kHeadDim
                      : p.cache + ((static_cast<size_t>(ri.x) * 2 + 1) * H + h) * static_cast<size_t>(p.seq_capacity) * kHeadDim;
    };

    if (warp < kProducers) {
        // ---- producers: stage sequence over (item, chunk); producer w owns the stages with index = w (mod 4) -----------
        if (lane == 0) {
            // No dependency wait here: the encoder K/V store never changes during decoding, and the cached
            // self-attention positions below t_u were written by earlier steps, which completed before this one began.
            long long st = 0;
            int item_no = 0;
            bool ok = true;
            long long last_issued = -1;
            for (int item = b; item < n_items && ok; item += G, ++item_no) {
                const int r = item / H, h = item % H;
                const int4 ri = p.row_info[r];
                const int len = item_len(ri);
                const int chunks = len > 0 ? (len + kStagePos - 1) / kStagePos : 1;
                const __nv_bfloat16 *kb = k_base(ri, h), *vb = v_base(ri, h);
                for (int c = 0; c < chunks; ++c, ++st) {
                    if (static_cast<int>(st % kProducers) != warp) continue;
                    const int s = static_cast<int>(st % kStages);
                    if (st >= kStages && !mbar_wait(&bar_empty[s], static_cast<uint32_t>((st / kStages) - 1) & 1, &abort_flag)) { ok = false; break; }
                    const int n_pos = min(kStagePos, len - c * kStagePos);
                    meta[s].q_slot = item_no % kQSlots;
                    meta[s].n_pos = n_pos > 0 ? n_pos : 0;
                    meta[s].first = c == 0;
                    meta[s].last = c == chunks - 1;
                    uint8_t *dst = ring + static_cast<size_t>(s) * kStageBytes;
                    if (n_pos > 0) {
                        const uint32_t bytes = static_cast<uint32_t>(n_pos) * 128u;
                        mbar_expect_tx(&bar_full[s], 2 * bytes);
                        bulk_load(dst, kb + static_cast<size_t>(c) * kStagePos * kHeadDim, bytes, &bar_full[s]);
                        bulk_load(dst + kStagePos * 128, vb + static_cast<size_t>(c) * kStagePos * kHeadDim, bytes, &bar_full[s]);
                    } else {
                        mbar_arrive(&bar_full[s]);          // an item without cached positions still owns one (empty) stage
                    }
                    last_issued = st;
                }
            }
            if (!ok && last_issued >= 0) {
                const long long start = clock64();
                while (!mbar_try_wait(&bar_full[last_issued % kStages], static_cast<uint32_t>(last_issued / kStages) & 1) &&
                       clock64() - start < kWaitCycles / 8) {}
            }
        }
    } else if (warp == kProducers) {
        // ---- query warp: q = rstd * (raw - mean * c1) + c2, scaled; self: also the appended key and value -------------------
        // Four items at a time, one per group of eight lanes (a lane holds 8 of the 64 head dimensions), so that the
        // global-memory latency of one item's operands is shared by four.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int d_model = H * kHeadDim;
        const int grp = lane >> 3, sub = lane & 7;
        bool ok = true;
        for (int base_no = 0; ok; base_no += kQSlots) {
            const int item_no = base_no + grp;
            const long long item = static_cast<long long>(b) + static_cast<long long>(item_no) * G;
            if (static_cast<long long>(b) + static_cast<long long>(base_no) * G >= n_items) break;
            if (item < n_items) {
                const int r = static_cast<int>(item / H), h = static_cast<int>(item % H);
                const int slot = grp;                   // = item_no % kQSlots
                if (item_no >= kQSlots) ok = mbar_wait(&bar_q_empty[slot], static_cast<uint32_t>((item_no / kQSlots) - 1) & 1, &abort_flag);
                if (ok) {
                    const float2 st = p.ln_stats ? p.ln_stats[r] : make_float2(0.f, 1.f);
                    const int4 ri = p.row_info[r];
                    const int n_vec = kCross ? 1 : 3;          // q, and for self-attention k and v of the new position
                    float y[3][8], c1[3][8], c2[3][8];
#pragma unroll
                    for (int v = 0; v < 3; ++v) {
                        if (v >= n_vec) continue;
                        const int col = v * d_model + h * kHeadDim + sub * 8;
                        load8(p.q + static_cast<size_t>(r) * p.ldq + col, y[v]);
                        if (p.ln_stats) { load8(p.ln_c1 + col, c1[v]); load8(p.ln_c2 + col, c2[v]); }
                    }
#pragma unroll
                    for (int v = 0; v < 3; ++v) {
                        if (v >= n_vec) continue;
                        if (p.ln_stats) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) y[v][e] = fmaf(st.y, y[v][e] - st.x * c1[v][e], c2[v][e]);
                        }
                        if (v == 0) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) q_s[slot][sub * 8 + e] = y[0][e] * p.scale;
                        } else {
                            Raw8<__nv_bfloat16> packed;            // rounded to bf16, as the cache stores it
                            packed.set(y[v]);
                            __nv_bfloat16 *dst = const_cast<__nv_bfloat16 *>(v == 1 ? k_base(ri, h) : v_base(ri, h)) + static_cast<size_t>(ri.y) * kHeadDim + sub * 8;
                            packed.store(dst);
                            float back[8];
                            packed.get(back);
#pragma unroll
                            for (int e = 0; e < 8; ++e) (v == 1 ? new_k : new_v)[slot][sub * 8 + e] = back[e];
                        }
                    }
                }
            }
            __syncwarp();
            if (ok && item < n_items && sub == 0) mbar_arrive(&bar_q_full[grp]);
            ok = __all_sync(0xffffffffu, ok);
        }
    } else if (warp == kProducers + 1) {
        // ---- merge warp: combine the consumer warps' partials of a finished item, write the output row --------------------
        int item_no = 0;
        bool ok = true;
        for (int item = b; item < n_items && ok; item += G, ++item_no) {
            const int slot = item_no % kMergeSlots;
            ok = mbar_wait(&bar_m_full[slot], static_cast<uint32_t>(item_no / kMergeSlots) & 1, &abort_flag);
            if (!ok) break;
            const int r = item / H, h = item % H;
            float big = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsumers; ++w) big = fmaxf(big, mg_m[slot][w]);
            float lsum = 0.f, a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumers; ++w) {
                const float wgt = (mg_m[slot][w] == -INFINITY) ? 0.f : expf(mg_m[slot][w] - big);
                lsum = fmaf(mg_l[slot][w], wgt, lsum);
                a0 = fmaf(mg_acc[slot][w][2 * lane], wgt, a0);
                a1 = fmaf(mg_acc[slot][w][2 * lane + 1], wgt, a1);
            }
            const float inv = 1.f / lsum;
            *reinterpret_cast<float2 *>(p.out + static_cast<size_t>(r) * p.ldo + h * kHeadDim + 2 * lane) = make_float2(a0 * inv, a1 * inv);
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_m_empty[slot]);
        }
    } else {
        // ---- consumers: warp cw takes positions kPosPerWarp * cw .. + kPosPerWarp - 1 of every stage -------------------------
        const int cw = warp - kProducers - 2;
        const int dg = lane & 7, pg = lane >> 3;
        long long st = 0;
        int item_no = 0;
        bool ok = true;
        for (int item = b; item < n_items && ok; item += G, ++item_no) {
            float m = -INFINITY, l = 0.f, acc[8], qv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            const int q_slot = item_no % kQSlots;
            ok = mbar_wait(&bar_q_full[q_slot], static_cast<uint32_t>(item_no / kQSlots) & 1, &abort_flag);
            if (!ok) break;
#pragma unroll
            for (int i = 0; i < 8; ++i) qv[i] = q_s[q_slot][dg * 8 + i];
            bool last = false;
            while (!last && ok) {
                const int s = static_cast<int>(st % kStages);
                ok = mbar_wait(&bar_full[s], static_cast<uint32_t>(st / kStages) & 1, &abort_flag);
                if (!ok) break;
                const StageMeta mt = meta[s];
                last = mt.last != 0;
                const uint8_t *kt = ring + static_cast<size_t>(s) * kStageBytes, *vt = kt + kStagePos * 128;
                const int p0 = cw * kPosPerWarp;
                if (p0 < mt.n_pos) {
                    float sc[kPosIters], cmax = -INFINITY;
                    uint4 vraw[kPosIters];
#pragma unroll
                    for (int i = 0; i < kPosIters; ++i) {
                        const int pos = p0 + i * 4 + pg;
                        float d = 0.f;
                        if (pos < mt.n_pos) {
                            const uint4 kr = *reinterpret_cast<const uint4 *>(kt + pos * 128 + dg * 16);
                            vraw[i] = *reinterpret_cast<const uint4 *>(vt + pos * 128 + dg * 16);
                            const uint32_t w[4] = {kr.x, kr.y, kr.z, kr.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                d = fmaf(qv[2 * j], __uint_as_float(w[j] << 16), d);
                                d = fmaf(qv[2 * j + 1], __uint_as_float(w[j] & 0xFFFF0000u), d);
                            }
                        } else vraw[i] = make_uint4(0u, 0u, 0u, 0u);
                        d += __shfl_xor_sync(0xffffffffu, d, 1);
                        d += __shfl_xor_sync(0xffffffffu, d, 2);
                        d += __shfl_xor_sync(0xffffffffu, d, 4);
                        sc[i] = pos < mt.n_pos ? d : -INFINITY;
                        cmax = fmaxf(cmax, sc[i]);
                    }
                    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
                    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
                    const float m_new = fmaxf(m, cmax);
                    const float corr = expf(m - m_new);
                    l *= corr;
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[j] *= corr;
#pragma unroll
                    for (int i = 0; i < kPosIters; ++i) {
                        const float pr = expf(sc[i] - m_new);
                        const uint32_t w[4] = {vraw[i].x, vraw[i].y, vraw[i].z, vraw[i].w};
                        l += pr;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            acc[2 * j] = fmaf(pr, __uint_as_float(w[j] << 16), acc[2 * j]);
                            acc[2 * j + 1] = fmaf(pr, __uint_as_float(w[j] & 0xFFFF0000u), acc[2 * j + 1]);
                        }
                    }
                    m = m_new;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_empty[s]);
                ++st;
            }
            if (!ok) break;
            if (!kCross && cw == kConsumers - 1) {
                // the position this step appends: key and value prepared by the query warp (position group 0 only)
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qv[i], new_k[q_slot][dg * 8 + i], d);
                d += __shfl_xor_sync(0xffffffffu, d, 1);
                d += __shfl_xor_sync(0xffffffffu, d, 2);
                d += __shfl_xor_sync(0xffffffffu, d, 4);
                const float m_new = fmaxf(m, d);
                const float corr = expf(m - m_new), pr = pg == 0 ? expf(d - m_new) : 0.f;
                l = l * corr + pr;
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = fmaf(pr, new_v[q_slot][dg * 8 + i], acc[i] * corr);
                m = m_new;
            }
            // the four position groups share m: sum them, then hand the partial to the merge warp
            l += __shfl_xor_sync(0xffffffffu, l, 8);
            l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 8);
                acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 16);
            }
            const int ms = item_no % kMergeSlots;
            if (item_no >= kMergeSlots) ok = mbar_wait(&bar_m_empty[ms], static_cast<uint32_t>((item_no / kMergeSlots) - 1) & 1, &abort_flag);
            if (!ok) break;
            if (lane == 0) { mg_m[ms][cw] = m; mg_l[ms][cw] = l; }
            if (pg == 0) {
#pragma unroll
                for (int j = 0; j < 8; ++j) mg_acc[ms][cw][dg * 8 + j] = acc[j];
            }
            __syncwarp();
            if (lane == 0) { mbar_arrive(&bar_m_full[ms]); mbar_arrive(&bar_q_empty[q_slot]); }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&p.err_state->error, kErrTimeout);
}

}  // namespace as
}  // namespace aed
