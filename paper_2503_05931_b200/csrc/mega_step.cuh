// Persistent decode-step kernel for small batches (bf16 mode, at most kMaxRows active rows).
//
// One launch runs all layers of a decoding step.  The grid is one thread block per SM, all resident at once.
// A step with few rows is a chain of dependent stages whose arithmetic is tiny: what it costs is the latency of
// every hand-over between stages and the time until a stage's weights are on chip.  So
//   * every block owns, for the whole step, a fixed share of every weight matrix, and four producer threads
//     stream that share through one ring of 16 KB shared-memory slots, running ahead of the arithmetic across
//     stage and layer boundaries (weights are static: a producer waits for free slots only);
//   * a layer is five stages instead of eight kernels:
//       S1  [q|k|v]_raw += (gamma1 * x) Wqkv^T                         tiles (128 features x 64 k), split-K
//       S2  per (head, row block): LayerNorm fold, cache append, self-attention, x += o Wo[:, head]^T
//       S3  per (head, row block): LayerNorm of its rows, q' = LN2(x) Wqc[head]^T, cross-attention over the
//           rows' own encoder frames, x_next = x + o' Woc[:, head]^T
//       S4  hidden_raw += (gamma3 * x) W1^T                             tiles, split-K
//       S5  x += relu(LN3-corrected hidden) W2^T                        tiles, split-K
//     handed over through arrival counters in global memory (release / acquire at GPU scope) that every block
//     polls with a bounded wait;
//   * the arithmetic is warp-level mma.sync (m16n8k16, bf16 x bf16 -> fp32) straight from the swizzled tiles the
//     TMA unit wrote, activations as a bf16 high plane plus a bf16 low plane (value - high): no accumulator
//     round trip through tensor memory, no transposition, partial sums leave as 8-byte red.global.
// LayerNorm is folded as in the projection kernel: LN(x) W^T = rstd * ((gamma*x) W^T - mean * c1) + c2.
//
// Buffers written by one block and read by another (x, [q|k|v], hidden, statistics) are only ever read with
// ld.global.cg, so no stale line can sit in an L1 cache.  The residual stream alternates between two buffers:
// S3 reads its rows from one and accumulates x_next into the other (cleared two stages earlier), because blocks
// of the same row block read and write those rows without a hand-over in between.
//
// A wait that runs out raises the abort word: from then on every wait in every block returns at once, the step
// runs to its end on whatever data it has, and the host reports AED_ERR_TIMEOUT.
#pragma once
#include "step_gemm.cuh"
#include "step_kernels.cuh"

namespace aed {
namespace mega {

using namespace tc;

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kProducerWarps = 4;       // one issuing thread each: a thread's bulk copies complete one at a time
constexpr int kThreads = (kConsumerWarps + kProducerWarps) * 32;
constexpr int kSlotBytes = 16384;       // 128 weight rows x 64 k (bf16), or two boxes of 64 rows x 64 k
constexpr int kMaxSlots = 12;
constexpr int kMaxRows = 64;            // active rows of a step on this path
constexpr int kUnitRows = 8;            // rows one (head, row block) unit holds
constexpr int kStagesPerLayer = 5;

struct LayerArgs {
    const __nv_bfloat16 *ln1_g, *ln2_g, *ln3_g;
    const float *c1_qkv, *c2_qkv, *c1_qc, *c2_qc, *c1_ff, *c2_ff;       // LayerNorm-fold constants
    const __nv_bfloat16 *b_o, *b_oc, *b_ff2;                             // nullable
    __nv_bfloat16 *self_cache;                                           // [batch][2][H][max_dec_len][64]
    const __nv_bfloat16 *cross;                                          // [2][H][frame_capacity][64]
};

struct MegaParams {
    int n_layers, d, n_heads, d_ffn;
    int n_slots;
    int self_capacity, frame_capacity;
    float scale, eps;
    float *x0, *x1;             // residual stream: layer l reads x(l & 1) and leaves its result in x((l + 1) & 1)
    float *qkv, *hid;           // [rows, 3d], [rows, F] split-K accumulators
    float2 *stats1, *stats3;    // (mean, rstd) per row for LN1 and LN3
    const int4 *row_info;       // (utterance, t_u, encoder length, encoder offset) per compact row
    DecState *state;
    int *bars;                  // [n_layers * 5] arrival counters followed by the abort word
    const CUtensorMap *maps;    // [n_layers][6]: w_qkv, w_o, w_q_c (64-row boxes), w_o_c, w_ff1, w_ff2
    const LayerArgs *layers;    // [n_layers]
};

// Shared-memory carve-up (after the ring), identical on host and device.
struct SmemLayout {
    int ring, planes, scratch, q_s, o_planes, merge, rows, total;
};
__host__ __device__ inline SmemLayout smem_layout(int n_slots)
{
    SmemLayout s;
    int off = 0;
    s.ring = off; off += n_slots * kSlotBytes;
    s.planes = off; off += 32768;             // two 16 KB activation tiles (tile stages) / LN2 planes of 8 rows x d
    s.scratch = off; off += 16384;            // per-warp partial queries [8][8][64] fp32; block reductions
    s.q_s = off; off += kUnitRows * 64 * 4;
    s.o_planes = off; off += 2 * kUnitRows * 128;
    s.merge = off; off += (kConsumerWarps * 2 + kConsumerWarps * 64) * 4;
    s.rows = off; off += kUnitRows * (16 + 4 + 8);   // row table entries, global row index, (mean, rstd)
    s.total = off;
    return s;
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

__device__ __forceinline__ float4 ldcg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ void load8_cg(const float *p, float (&v)[8])
{
    const float4 a = ldcg4(p), b = ldcg4(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void red_add_v2(float *addr, float a, float b)
{
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t &r0, uint32_t &r1)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
// D += A (16 x 16, row) * B (16 x 8, col), bf16 operands, fp32 accumulation
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte offset of (row, 16-byte chunk) in a tile of 128-byte rows with the 128-byte swizzle (what TMA writes and
// what the activation planes use too).
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return static_cast<uint32_t>(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// What one block does in a layer: fixed at launch, the same for the producers and the consumers.
struct Schedule {
    int s1_begin, s1_end, s4_begin, s4_end, s5_begin, s5_end;   // linear tile ranges (feature tile major)
    int kb_d, kb_f;             // k-blocks of d_model and of d_ffn
    bool unit;                  // this block is a (head, row block) unit
    int head, rb, n_rb;
    int n_o;                    // 128-feature slots of an output projection slice
    int n_qc;                   // slots of a cross-query slice (two k-blocks each)
    __device__ int slots_per_layer() const
    {
        return (s1_end - s1_begin) + (s4_end - s4_begin) + (s5_end - s5_begin) + (unit ? 2 * n_o + n_qc : 0);
    }
};
__device__ inline Schedule make_schedule(const MegaParams &p)
{
    Schedule s;
    const int G = gridDim.x, c = blockIdx.x;
    s.kb_d = p.d / kBlockK;
    s.kb_f = p.d_ffn / kBlockK;
    const long long t1 = static_cast<long long>((3 * p.d + kTileM - 1) / kTileM) * s.kb_d;
    const long long t4 = static_cast<long long>((p.d_ffn + kTileM - 1) / kTileM) * s.kb_d;
    const long long t5 = static_cast<long long>((p.d + kTileM - 1) / kTileM) * s.kb_f;
    s.s1_begin = static_cast<int>(t1 * c / G); s.s1_end = static_cast<int>(t1 * (c + 1) / G);
    s.s4_begin = static_cast<int>(t4 * c / G); s.s4_end = static_cast<int>(t4 * (c + 1) / G);
    s.s5_begin = static_cast<int>(t5 * c / G); s.s5_end = static_cast<int>(t5 * (c + 1) / G);
    s.n_rb = G / p.n_heads;
    s.unit = c < p.n_heads * s.n_rb;
    s.head = c / s.n_rb;
    s.rb = c % s.n_rb;
    s.n_o = (p.d + kTileM - 1) / kTileM;
    s.n_qc = (s.kb_d + 1) / 2;
    return s;
}

struct Ctx {
    uint8_t *ring, *planes, *scratch, *o_planes;
    float *q_s, *mg_m, *mg_l, *mg_acc;
    int4 *rows_s;
    int *grow_s;
    float2 *ln_s;
    uint64_t *full, *empty;
    volatile int *abort_flag;       // shared memory
    int *bars;                      // global arrival counters; bars[n_bars] is the abort word
    int n_bars;
    DecState *state;
    int n_slots;
    uint32_t q;                     // slots consumed so far
    int tid, warp, lane;
};

__device__ __forceinline__ bool slot_wait(Ctx &c)
{
    const uint32_t s = c.q % c.n_slots;
    return mbar_wait(&c.full[s], (c.q / c.n_slots) & 1, c.abort_flag);
}
__device__ __forceinline__ uint8_t *slot_ptr(const Ctx &c) { return c.ring + static_cast<size_t>(c.q % c.n_slots) * kSlotBytes; }
__device__ __forceinline__ void slot_release(Ctx &c)
{
    __syncwarp();
    if (c.lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&c.empty[c.q % c.n_slots])) : "memory");
    ++c.q;
}

// Every consumer thread has finished its global writes of the stage: publish them.
__device__ __forceinline__ void grid_arrive(Ctx &c, int idx)
{
    consumer_sync();
    if (c.tid == 0) {
        __threadfence();
        atomicAdd(&c.bars[idx], 1);
    }
}
// All blocks have published stage idx.
__device__ __forceinline__ void grid_wait(Ctx &c, int idx)
{
    if (c.tid == 0) {
        const int *bar = c.bars + idx, *abort_word = c.bars + c.n_bars;
        const int expected = gridDim.x;
        bounded_poll([&] { return ld_acquire(bar) >= expected || ld_acquire(abort_word) != 0; }, [] { return clock64(); },
                     kWaitCycles, c.abort_flag);
        if (ld_acquire(abort_word) != 0) *c.abort_flag = 1;
        if (*c.abort_flag) {                 // tell every other block, and the host
            atomicExch(c.bars + c.n_bars, 1);
            atomicExch(&c.state->error, kErrTimeout);
        }
    }
    consumer_sync();
}

// ---- tile stages (S1, S4, S5) -------------------------------------------------------------------------------------
enum TileMode { T_GAMMA = 0, T_LN_RELU = 1 };

struct TileArgs {
    const float *src; int ld_src;               // activation source [rows, ld_src] fp32
    const __nv_bfloat16 *gamma;                 // T_GAMMA
    const float *c1, *c2; const float2 *stats;  // T_LN_RELU
    float *out; int ldo; int n_features;
    const __nv_bfloat16 *bias;                  // added with the k-block 0 tile of a feature tile; nullable
};

template <int MODE>
__device__ void tile_stage(Ctx &c, int begin, int end, int KB, const TileArgs &a, int n)
{
    const int mt = (n + 15) >> 4;               // 16-row MMA tiles
    const int rows_pad = mt << 4;
    const int g = c.lane >> 2, t4 = c.lane & 3;
    float acc[4][2][4];
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[m][j][e] = 0.f;
    int cur_ft = -1;
    bool with_bias = false;

    auto flush = [&](int ft) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            if (m >= mt) continue;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int f = ft * kTileM + 16 * c.warp + 8 * j + 2 * t4;
                if (f >= a.n_features) continue;
                float b0 = 0.f, b1 = 0.f;
                if (with_bias && a.bias) { b0 = to_f32(a.bias[f]); b1 = to_f32(a.bias[f + 1]); }
                const int r0 = 16 * m + g, r1 = r0 + 8;
                if (r0 < n) red_add_v2(a.out + static_cast<size_t>(r0) * a.ldo + f, acc[m][j][0] + b0, acc[m][j][1] + b1);
                if (r1 < n) red_add_v2(a.out + static_cast<size_t>(r1) * a.ldo + f, acc[m][j][2] + b0, acc[m][j][3] + b1);
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[m][j][e] = 0.f;
            }
        }
    };

    for (int i = begin; i < end; ++i) {
        const int ft = i / KB, kb = i - ft * KB;
        if (ft != cur_ft) {
            if (cur_ft >= 0) flush(cur_ft);
            cur_ft = ft;
            with_bias = false;
        }
        if (kb == 0) with_bias = true;
        // activation tile of this k-block: high plane, low plane, 64 rows x 128 B each, swizzled
        uint8_t *hi_tile = c.planes + ((i - begin) & 1) * 16384, *lo_tile = hi_tile + 8192;
        {
            const int ch = c.tid & 7, rbase = c.tid >> 3;
            const int k = kb * kBlockK + ch * 8;
            float gm[8], c1[8], c2[8];
            if (MODE == T_GAMMA) load8(a.gamma + k, gm);
            if (MODE == T_LN_RELU) { load8(a.c1 + k, c1); load8(a.c2 + k, c2); }
            for (int rl = rbase; rl < rows_pad; rl += 32) {
                float y[8];
                if (rl < n) {
                    load8_cg(a.src + static_cast<size_t>(rl) * a.ld_src + k, y);
                    if (MODE == T_GAMMA) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] *= gm[e];
                    } else {
                        const float2 st = __ldcg(a.stats + rl);
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] = fmaxf(fmaf(st.y, y[e] - st.x * c1[e], c2[e]), 0.f);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) y[e] = 0.f;
                }
                uint4 hi, lo;
                sg::split_planes(y, hi, lo);
                const uint32_t off = swz(rl, ch);
                *reinterpret_cast<uint4 *>(hi_tile + off) = hi;
                *reinterpret_cast<uint4 *>(lo_tile + off) = lo;
            }
        }
        consumer_sync();
        slot_wait(c);
        {
            const uint32_t wt = smem_u32(slot_ptr(c)), ph = smem_u32(hi_tile), pl = smem_u32(lo_tile);
            // B fragments: this warp's 16 features, all four k-steps
            uint32_t bf[2][4][2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int row = 16 * c.warp + 8 * j + (c.lane & 7);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t r[4];
                    ldmatrix_x4(wt + swz(row, 4 * half + (c.lane >> 3)), r);
                    bf[j][2 * half][0] = r[0]; bf[j][2 * half][1] = r[1];
                    bf[j][2 * half + 1][0] = r[2]; bf[j][2 * half + 1][1] = r[3];
                }
            }
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                if (m >= mt) continue;
                const int row = 16 * m + (c.lane & 7) + ((c.lane >> 3) & 1) * 8;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t ah[4], al[4];
                    const uint32_t off = swz(row, 2 * ks + (c.lane >> 4));
                    ldmatrix_x4(ph + off, ah);
                    ldmatrix_x4(pl + off, al);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        mma_16816(acc[m][j], ah[0], ah[1], ah[2], ah[3], bf[j][ks][0], bf[j][ks][1]);
                        mma_16816(acc[m][j], al[0], al[1], al[2], al[3], bf[j][ks][0], bf[j][ks][1]);
                    }
                }
            }
        }
        slot_release(c);
    }
    if (cur_ft >= 0) flush(cur_ft);
}

// (mean, rstd) of row r of src [rows, d], by all consumer threads of the block.
__device__ void row_stats(Ctx &c, const float *src, int r, int d, float eps, float2 *out)
{
    float *red = reinterpret_cast<float *>(c.scratch);
    const float *xr = src + static_cast<size_t>(r) * d;
    float s = 0.f;
    for (int i = c.tid * 4; i < d; i += kConsumerThreads * 4) {
        const float4 v = ldcg4(xr + i);
        s += (v.x + v.y) + (v.z + v.w);
    }
    s = warp_sum(s);
    if (c.lane == 0) red[c.warp] = s;
    consumer_sync();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) tot += red[w];
    const float mean = tot / d;
    float q = 0.f;
    for (int i = c.tid * 4; i < d; i += kConsumerThreads * 4) {
        const float4 v = ldcg4(xr + i);
        const float d0 = v.x - mean, d1 = v.y - mean, d2 = v.z - mean, d3 = v.w - mean;
        q += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
    }
    q = warp_sum(q);
    if (c.lane == 0) red[kConsumerWarps + c.warp] = q;
    consumer_sync();
    float qt = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) qt += red[kConsumerWarps + w];
    if (c.tid == 0) *out = make_float2(mean, rsqrtf(qt / d + eps));
    consumer_sync();        // the reduction buffer is free again
}

// Clear count floats (a multiple of 4) of buf, spread over the whole grid.
__device__ __forceinline__ void zero_floats(const Ctx &c, float *buf, size_t count)
{
    float4 *z = reinterpret_cast<float4 *>(buf);
    const size_t n4 = count / 4;
    for (size_t i = static_cast<size_t>(blockIdx.x) * kConsumerThreads + c.tid; i < n4; i += static_cast<size_t>(gridDim.x) * kConsumerThreads)
        z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// ---- unit stages (S2, S3) -----------------------------------------------------------------------------------------

// Flash-decoding attention of the unit's rows for one head.  The eight consumer warps are shared out over the rows
// (a power-of-two number of warps per row); the warps of a row take alternating 16-position chunks, keep a running
// (max, sum, accumulator) and are merged through shared memory.  Lanes: 8 dimension groups x 4 position groups; a
// lane's 4 keys and 4 values of a chunk (16 bytes each) are requested together, the next chunk before the current
// one is reduced.  Queries come from q_s (already scaled).  kSelf: the position this step appends is taken from
// the projection output (with the LayerNorm fold applied), stored to the cache and attended to.
// Result: the rows' outputs as bf16 high/low planes in o_planes (8 rows x 64, swizzled).
template <bool kSelf>
__device__ void attend_rows(Ctx &c, const MegaParams &p, const LayerArgs &la, int head, int nr)
{
    typedef __nv_bfloat16 CT;
    int nr_pad = 1;
    while (nr_pad < nr) nr_pad <<= 1;
    const int wpr = kConsumerWarps / nr_pad;
    const int li = c.warp / wpr, part = c.warp % wpr;
    const int dg = c.lane & 7, pg = c.lane >> 3;
    float m = -INFINITY, l = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    if (li < nr) {
        const int4 ri = c.rows_s[li];
        const int len = kSelf ? ri.y + 1 : ri.z;
        const int len_static = kSelf ? len - 1 : len;
        const CT *kbase, *vbase;
        if (kSelf) {
            kbase = la.self_cache + ((static_cast<size_t>(ri.x) * 2 + 0) * p.n_heads + head) * static_cast<size_t>(p.self_capacity) * kHeadDim;
            vbase = la.self_cache + ((static_cast<size_t>(ri.x) * 2 + 1) * p.n_heads + head) * static_cast<size_t>(p.self_capacity) * kHeadDim;
        } else {
            kbase = la.cross + (static_cast<size_t>(0 * p.n_heads + head) * p.frame_capacity + ri.w) * kHeadDim;
            vbase = la.cross + (static_cast<size_t>(1 * p.n_heads + head) * p.frame_capacity + ri.w) * kHeadDim;
        }
        Raw8<CT> rk[4], rv[4], nk[4], nv[4], new_k, new_v;
        auto load_chunk = [&](int p0, Raw8<CT>(&k4)[4], Raw8<CT>(&v4)[4]) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int pos = p0 + i * 4 + pg;
                if (pos < len_static) {
                    k4[i].load(kbase + static_cast<size_t>(pos) * kHeadDim + dg * 8);
                    v4[i].load(vbase + static_cast<size_t>(pos) * kHeadDim + dg * 8);
                } else { k4[i].zero(); v4[i].zero(); }
            }
        };
        const int step = wpr * kFusedChunk;
        load_chunk(part * kFusedChunk, rk, rv);
        const int new_chunk = (len - 1) / kFusedChunk;
        const bool owns_new = kSelf && part == new_chunk % wpr;
        if (owns_new) {
            // key and value of the new position: raw projection output with the LayerNorm fold applied
            const int r = c.grow_s[li];
            const float2 st = c.ln_s[li];
            const int col = head * kHeadDim + dg * 8;
            float kn[8], vn[8], c1[8], c2[8];
            load8_cg(p.qkv + static_cast<size_t>(r) * 3 * p.d + p.d + col, kn);
            load8(la.c1_qkv + p.d + col, c1); load8(la.c2_qkv + p.d + col, c2);
#pragma unroll
            for (int i = 0; i < 8; ++i) kn[i] = fmaf(st.y, kn[i] - st.x * c1[i], c2[i]);
            load8_cg(p.qkv + static_cast<size_t>(r) * 3 * p.d + 2 * p.d + col, vn);
            load8(la.c1_qkv + 2 * p.d + col, c1); load8(la.c2_qkv + 2 * p.d + col, c2);
#pragma unroll
            for (int i = 0; i < 8; ++i) vn[i] = fmaf(st.y, vn[i] - st.x * c1[i], c2[i]);
            new_k.set(kn);
            new_v.set(vn);
            if (pg == 0) {      // append; nobody else reads this position during the step
                new_k.store(const_cast<CT *>(kbase) + static_cast<size_t>(len - 1) * kHeadDim + dg * 8);
                new_v.store(const_cast<CT *>(vbase) + static_cast<size_t>(len - 1) * kHeadDim + dg * 8);
            }
        }
        float qv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) qv[i] = c.q_s[li * kHeadDim + dg * 8 + i];
        for (int p0 = part * kFusedChunk; p0 < len; p0 += step) {
            if (p0 + step < len) load_chunk(p0 + step, nk, nv);
            if (owns_new && p0 == new_chunk * kFusedChunk) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (p0 + i * 4 + pg == len - 1) { rk[i] = new_k; rv[i] = new_v; }
            }
            float s[4], cmax = -INFINITY;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float kf[8], d = 0.f;
                rk[i].get(kf);
#pragma unroll
                for (int j = 0; j < 8; ++j) d = fmaf(qv[j], kf[j], d);
                d += __shfl_xor_sync(0xffffffffu, d, 1);
                d += __shfl_xor_sync(0xffffffffu, d, 2);
                d += __shfl_xor_sync(0xffffffffu, d, 4);
                s[i] = (p0 + i * 4 + pg < len) ? d : -INFINITY;
                cmax = fmaxf(cmax, s[i]);
            }
            cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
            cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));     // finite: the chunk holds a valid position
            const float m_new = fmaxf(m, cmax);
            const float corr = expf(m - m_new);
            l *= corr;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] *= corr;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float pr = expf(s[i] - m_new);
                float vf[8];
                rv[i].get(vf);
                l += pr;
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] = fmaf(pr, vf[j], acc[j]);
            }
            m = m_new;
#pragma unroll
            for (int i = 0; i < 4; ++i) { rk[i] = nk[i]; rv[i] = nv[i]; }
        }
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 8);
            acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 16);
        }
    }
    if (c.lane == 0) { c.mg_m[c.warp] = m; c.mg_l[c.warp] = l; }
    if (pg == 0) {
#pragma unroll
        for (int j = 0; j < 8; ++j) c.mg_acc[c.warp * kHeadDim + dg * 8 + j] = acc[j];
    }
    consumer_sync();
    // merge the warps of each row; thread -> (row, dimension)
    for (int e = c.tid; e < kUnitRows * kHeadDim; e += kConsumerThreads) {
        const int row = e / kHeadDim, dim = e % kHeadDim;
        float o = 0.f;
        if (row < nr) {
            float big = -INFINITY;
            for (int w = row * wpr; w < (row + 1) * wpr; ++w) big = fmaxf(big, c.mg_m[w]);
            float lsum = 0.f, a = 0.f;
            for (int w = row * wpr; w < (row + 1) * wpr; ++w) {
                const float wgt = (c.mg_m[w] == -INFINITY) ? 0.f : expf(c.mg_m[w] - big);
                lsum = fmaf(c.mg_l[w], wgt, lsum);
                a = fmaf(c.mg_acc[w * kHeadDim + dim], wgt, a);
            }
            o = a / lsum;
        }
        const __nv_bfloat16 hi = __float2bfloat16_rn(o);
        const __nv_bfloat16 lo = __float2bfloat16_rn(o - __bfloat162float(hi));
        const uint32_t off = swz(row, dim >> 3) + (dim & 7) * 2;
        *reinterpret_cast<__nv_bfloat16 *>(c.o_planes + off) = hi;
        *reinterpret_cast<__nv_bfloat16 *>(c.o_planes + kUnitRows * 128 + off) = lo;
    }
    consumer_sync();
}

// x_out[rows of the unit] += o Wo[:, head]^T (+ bias and, when x_in is given, x_in: by the block of head 0).
// The slice arrives as n_o slots of 128 output features x 64 k.
__device__ void out_projection(Ctx &c, const MegaParams &p, int n_o, int nr, bool first_head, const __nv_bfloat16 *bias,
                               const float *x_in, float *x_out)
{
    const int g = c.lane >> 2, t4 = c.lane & 3;
    const uint32_t oh = smem_u32(c.o_planes), ol = oh + kUnitRows * 128;
    uint32_t ah[4][2], al[4][2];
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
        const uint32_t off = swz(c.lane & 7, 2 * ks + ((c.lane >> 3) & 1));
        ldmatrix_x2(oh + off, ah[ks][0], ah[ks][1]);
        ldmatrix_x2(ol + off, al[ks][0], al[ks][1]);
    }
    const int r = g < nr ? c.grow_s[g] : 0;
    for (int j = 0; j < n_o; ++j) {
        slot_wait(c);
        const uint32_t wt = smem_u32(slot_ptr(c));
        float acc[2][4];
#pragma unroll
        for (int jb = 0; jb < 2; ++jb) {
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[jb][e] = 0.f;
            const int row = 16 * c.warp + 8 * jb + (c.lane & 7);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t b[4];
                ldmatrix_x4(wt + swz(row, 4 * half + (c.lane >> 3)), b);
                mma_16816(acc[jb], ah[2 * half][0], 0u, ah[2 * half][1], 0u, b[0], b[1]);
                mma_16816(acc[jb], al[2 * half][0], 0u, al[2 * half][1], 0u, b[0], b[1]);
                mma_16816(acc[jb], ah[2 * half + 1][0], 0u, ah[2 * half + 1][1], 0u, b[2], b[3]);
                mma_16816(acc[jb], al[2 * half + 1][0], 0u, al[2 * half + 1][1], 0u, b[2], b[3]);
            }
        }
        slot_release(c);
        if (g < nr) {
#pragma unroll
            for (int jb = 0; jb < 2; ++jb) {
                const int f = j * kTileM + 16 * c.warp + 8 * jb + 2 * t4;
                if (f >= p.d) continue;
                float v0 = acc[jb][0], v1 = acc[jb][1];
                if (first_head) {
                    if (bias) { v0 += to_f32(bias[f]); v1 += to_f32(bias[f + 1]); }
                    if (x_in) {
                        const float2 xi = __ldcg(reinterpret_cast<const float2 *>(x_in + static_cast<size_t>(r) * p.d + f));
                        v0 += xi.x; v1 += xi.y;
                    }
                }
                red_add_v2(x_out + static_cast<size_t>(r) * p.d + f, v0, v1);
            }
        }
    }
}

// The unit's rows of this step: row table entries and compact row indices into shared memory.  Returns their number.
__device__ __forceinline__ int load_unit_rows(Ctx &c, const MegaParams &p, const Schedule &s, int n)
{
    int nr = 0;
    if (s.unit && s.rb < n) nr = (n - s.rb + s.n_rb - 1) / s.n_rb;
    if (nr > kUnitRows) nr = kUnitRows;
    if (c.tid < kUnitRows) {
        const int r = s.rb + c.tid * s.n_rb;
        c.grow_s[c.tid] = r;
        c.rows_s[c.tid] = c.tid < nr ? p.row_info[r] : make_int4(-1, 0, 0, 0);
    }
    return nr;
}

__device__ void self_stage(Ctx &c, const MegaParams &p, const LayerArgs &la, const Schedule &s, int nr, float *x_cur)
{
    if (nr > 0) {
        // statistics of LN1 and the rows' queries: q = rstd * (raw - mean * c1) + c2, scaled
        if (c.tid < nr) c.ln_s[c.tid] = __ldcg(p.stats1 + c.grow_s[c.tid]);
        consumer_sync();
        for (int e = c.tid; e < nr * kHeadDim; e += kConsumerThreads) {
            const int li = e / kHeadDim, col = s.head * kHeadDim + e % kHeadDim;
            const float2 st = c.ln_s[li];
            const float raw = __ldcg(p.qkv + static_cast<size_t>(c.grow_s[li]) * 3 * p.d + col);
            c.q_s[e] = fmaf(st.y, raw - st.x * la.c1_qkv[col], la.c2_qkv[col]) * p.scale;
        }
        consumer_sync();
        attend_rows<true>(c, p, la, s.head, nr);
        out_projection(c, p, s.n_o, nr, s.head == 0, la.b_o, nullptr, x_cur);
    } else {
        for (int j = 0; j < s.n_o; ++j) { slot_wait(c); slot_release(c); }
    }
}

__device__ void cross_stage(Ctx &c, const MegaParams &p, const LayerArgs &la, const Schedule &s, int nr,
                            const float *x_cur, float *x_next)
{
    if (nr == 0) {
        for (int j = 0; j < s.n_qc + s.n_o; ++j) { slot_wait(c); slot_release(c); }
        return;
    }
    const int d = p.d;
    // LayerNorm statistics of the unit's rows (one warp per row) and gamma2 * x as bf16 planes:
    // per k-block 8 rows x 128 B, high planes first, then the low planes
    uint8_t *pl_hi = c.planes, *pl_lo = c.planes + 16384;
    if (c.warp < nr) {
        const float *xr = x_cur + static_cast<size_t>(c.grow_s[c.warp]) * d;
        float4 v[8];                         // d <= 1024: at most 8 float4 per lane
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = (c.lane + 32 * j) * 4;
            v[j] = k < d ? ldcg4(xr + k) : make_float4(0.f, 0.f, 0.f, 0.f);
            sum += (v[j].x + v[j].y) + (v[j].z + v[j].w);
        }
        const float mean = warp_sum(sum) / d;
        float q = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = (c.lane + 32 * j) * 4;
            if (k < d) {
                const float d0 = v[j].x - mean, d1 = v[j].y - mean, d2 = v[j].z - mean, d3 = v[j].w - mean;
                q += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
            }
        }
        const float rstd = rsqrtf(warp_sum(q) / d + p.eps);
        if (c.lane == 0) c.ln_s[c.warp] = make_float2(mean, rstd);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = (c.lane + 32 * j) * 4;
            if (k >= d) continue;
            float gm[4];
            load4(la.ln2_g + k, gm);
            const float y[4] = {v[j].x * gm[0], v[j].y * gm[1], v[j].z * gm[2], v[j].w * gm[3]};
            uint32_t h2[2], l2[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const __nv_bfloat16 h0 = __float2bfloat16_rn(y[2 * e]), h1 = __float2bfloat16_rn(y[2 * e + 1]);
                __nv_bfloat162 hp = __halves2bfloat162(h0, h1);
                h2[e] = *reinterpret_cast<uint32_t *>(&hp);
                l2[e] = sg::pack_bf16(y[2 * e] - __bfloat162float(h0), y[2 * e + 1] - __bfloat162float(h1));
            }
            const int kb = k >> 6, kk = k & 63;
            const uint32_t off = kb * 1024 + swz(c.warp, kk >> 3) + (kk & 7) * 2;
            *reinterpret_cast<uint2 *>(pl_hi + off) = make_uint2(h2[0], h2[1]);
            *reinterpret_cast<uint2 *>(pl_lo + off) = make_uint2(l2[0], l2[1]);
        }
    } else {
        // rows the unit does not have: zero planes, so that the MMA rows stay finite
        for (int kb = c.lane; kb < d / kBlockK; kb += 32) {
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                *reinterpret_cast<uint4 *>(pl_hi + kb * 1024 + swz(c.warp, ch)) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(pl_lo + kb * 1024 + swz(c.warp, ch)) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
    consumer_sync();
    // q'_raw = (gamma2 * x) Wqc[head]^T: warp w takes the slots w, w + 8, ... (two k-blocks each), partial sums
    // over its k-blocks for all 64 features, summed over the warps through shared memory
    {
        float acc[8][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
        const int kbs = d / kBlockK;
        for (int sl = 0; sl < s.n_qc; ++sl) {
            if (sl % kConsumerWarps == c.warp) {
                slot_wait(c);
                const uint32_t wt = smem_u32(slot_ptr(c));
                for (int b = 0; b < 2; ++b) {
                    const int kb = 2 * sl + b;
                    if (kb >= kbs) break;
                    const uint32_t wb = wt + b * 8192, ph = smem_u32(pl_hi) + kb * 1024, pl = smem_u32(pl_lo) + kb * 1024;
                    uint32_t ah[4][2], al[4][2];
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint32_t off = swz(c.lane & 7, 2 * ks + ((c.lane >> 3) & 1));
                        ldmatrix_x2(ph + off, ah[ks][0], ah[ks][1]);
                        ldmatrix_x2(pl + off, al[ks][0], al[ks][1]);
                    }
#pragma unroll
                    for (int nb = 0; nb < 8; ++nb) {
                        const int row = 8 * nb + (c.lane & 7);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t bb[4];
                            ldmatrix_x4(wb + swz(row, 4 * half + (c.lane >> 3)), bb);
                            mma_16816(acc[nb], ah[2 * half][0], 0u, ah[2 * half][1], 0u, bb[0], bb[1]);
                            mma_16816(acc[nb], al[2 * half][0], 0u, al[2 * half][1], 0u, bb[0], bb[1]);
                            mma_16816(acc[nb], ah[2 * half + 1][0], 0u, ah[2 * half + 1][1], 0u, bb[2], bb[3]);
                            mma_16816(acc[nb], al[2 * half + 1][0], 0u, al[2 * half + 1][1], 0u, bb[2], bb[3]);
                        }
                    }
                }
            }
            slot_release(c);
        }
        float *part = reinterpret_cast<float *>(c.scratch) + c.warp * (kUnitRows * kHeadDim);
        const int g = c.lane >> 2, t4 = c.lane & 3;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
            *reinterpret_cast<float2 *>(part + g * kHeadDim + 8 * nb + 2 * t4) = make_float2(acc[nb][0], acc[nb][1]);
    }
    consumer_sync();
    for (int e = c.tid; e < nr * kHeadDim; e += kConsumerThreads) {
        const int li = e / kHeadDim, col = s.head * kHeadDim + e % kHeadDim;
        float raw = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) raw += reinterpret_cast<const float *>(c.scratch)[w * (kUnitRows * kHeadDim) + e];
        const float2 st = c.ln_s[li];
        c.q_s[e] = fmaf(st.y, raw - st.x * la.c1_qc[col], la.c2_qc[col]) * p.scale;
    }
    consumer_sync();
    attend_rows<false>(c, p, la, s.head, nr);
    out_projection(c, p, s.n_o, nr, s.head == 0, la.b_oc, x_cur, x_next);
}

// ---- producers ------------------------------------------------------------------------------------------------

__device__ void produce(const MegaParams &p, const Schedule &s, uint8_t *ring, uint64_t *full, uint64_t *empty,
                        volatile int *abort_flag, int lane_id /* 0 .. kProducerWarps-1 */)
{
    uint32_t q = 0;
    bool ok = true;
    uint32_t last_mine = 0;
    bool issued_any = false;
    // one slot: `boxes` tensor boxes of box_bytes each, the second one k_step further along k
    auto issue = [&](const CUtensorMap *map, int k0, int row0, int box_bytes, int boxes, int k_step) {
        if (ok && static_cast<int>(q % kProducerWarps) == lane_id) {
            const uint32_t sl = q % p.n_slots;
            if (q >= static_cast<uint32_t>(p.n_slots)) ok = mbar_wait(&empty[sl], ((q / p.n_slots) - 1) & 1, abort_flag);
            if (ok) {
                uint8_t *dst = ring + static_cast<size_t>(sl) * kSlotBytes;
                mbar_expect_tx(&full[sl], box_bytes * boxes);
                tma_load_2d(dst, map, k0, row0, &full[sl]);
                if (boxes == 2) tma_load_2d(dst + box_bytes, map, k0 + k_step, row0, &full[sl]);
                last_mine = q;
                issued_any = true;
            }
        }
        ++q;
    };
    for (int l = 0; l < p.n_layers && ok; ++l) {
        const CUtensorMap *m = p.maps + 6 * l;
        for (int i = s.s1_begin; i < s.s1_end; ++i) issue(m + 0, (i % s.kb_d) * kBlockK, (i / s.kb_d) * kTileM, kSlotBytes, 1, 0);
        if (s.unit) {
            for (int j = 0; j < s.n_o; ++j) issue(m + 1, s.head * kHeadDim, j * kTileM, kSlotBytes, 1, 0);
            for (int sl = 0; sl < s.n_qc; ++sl) {
                const int kb = 2 * sl;
                issue(m + 2, kb * kBlockK, s.head * kHeadDim, kSlotBytes / 2, kb + 1 < s.kb_d ? 2 : 1, kBlockK);
            }
            for (int j = 0; j < s.n_o; ++j) issue(m + 3, s.head * kHeadDim, j * kTileM, kSlotBytes, 1, 0);
        }
        for (int i = s.s4_begin; i < s.s4_end; ++i) issue(m + 4, (i % s.kb_d) * kBlockK, (i / s.kb_d) * kTileM, kSlotBytes, 1, 0);
        for (int i = s.s5_begin; i < s.s5_end; ++i) issue(m + 5, (i % s.kb_f) * kBlockK, (i / s.kb_f) * kTileM, kSlotBytes, 1, 0);
    }
    if (!ok && issued_any) {
        // gave up: the copies this thread requested must land before the block's shared memory goes away
        const uint32_t first = last_mine >= static_cast<uint32_t>(p.n_slots) ? last_mine - p.n_slots + 1 : 0;
        for (uint32_t qq = first; qq <= last_mine; ++qq) {
            if (static_cast<int>(qq % kProducerWarps) != lane_id) continue;
            const long long start = clock64();
            while (!mbar_try_wait(&full[qq % p.n_slots], (qq / p.n_slots) & 1) && clock64() - start < kWaitCycles / 8) {}
        }
    }
}

// grid: one block per SM (all resident: the launch is cooperative).  Dynamic shared memory: smem_layout + 1024.
__global__ void __launch_bounds__(kThreads, 1) mega_step_kernel(const MegaParams p)
{
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t bar_full[kMaxSlots];
    __shared__ __align__(8) uint64_t bar_empty[kMaxSlots];
    __shared__ int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
    const SmemLayout lay = smem_layout(p.n_slots);
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_slots; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], kConsumerWarps); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const Schedule sched = make_schedule(p);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp >= kConsumerWarps) {
        if (lane == 0) produce(p, sched, base + lay.ring, bar_full, bar_empty, &abort_flag, warp - kConsumerWarps);
        return;
    }

    Ctx c;
    c.ring = base + lay.ring; c.planes = base + lay.planes; c.scratch = base + lay.scratch; c.o_planes = base + lay.o_planes;
    c.q_s = reinterpret_cast<float *>(base + lay.q_s);
    c.mg_m = reinterpret_cast<float *>(base + lay.merge); c.mg_l = c.mg_m + kConsumerWarps; c.mg_acc = c.mg_l + kConsumerWarps;
    c.rows_s = reinterpret_cast<int4 *>(base + lay.rows);
    c.grow_s = reinterpret_cast<int *>(base + lay.rows + kUnitRows * 16);
    c.ln_s = reinterpret_cast<float2 *>(base + lay.rows + kUnitRows * 20);
    c.full = bar_full; c.empty = bar_empty; c.abort_flag = &abort_flag;
    c.bars = p.bars; c.n_bars = p.n_layers * kStagesPerLayer; c.state = p.state;
    c.n_slots = p.n_slots; c.q = 0;
    c.tid = threadIdx.x; c.warp = warp; c.lane = lane;

    const int n = min(p.state->n_active, kMaxRows);
    const int d = p.d, F = p.d_ffn;
    const int nr = load_unit_rows(c, p, sched, n);
    consumer_sync();

    for (int l = 0; l < p.n_layers; ++l) {
        const LayerArgs la = p.layers[l];
        float *x_cur = (l & 1) ? p.x1 : p.x0, *x_next = (l & 1) ? p.x0 : p.x1;
        const int b0 = l * kStagesPerLayer;
        // S1: [q | k | v] raw; side jobs: LN1 statistics, clear the FFN accumulator and the next residual buffer
        if (l > 0) grid_wait(c, b0 - 1);
        if (static_cast<int>(blockIdx.x) < n) row_stats(c, x_cur, blockIdx.x, d, p.eps, p.stats1 + blockIdx.x);
        zero_floats(c, p.hid, static_cast<size_t>(n) * F);
        zero_floats(c, x_next, static_cast<size_t>(n) * d);
        {
            TileArgs a{};
            a.src = x_cur; a.ld_src = d; a.gamma = la.ln1_g;
            a.out = p.qkv; a.ldo = 3 * d; a.n_features = 3 * d; a.bias = nullptr;
            tile_stage<T_GAMMA>(c, sched.s1_begin, sched.s1_end, sched.kb_d, a, n);
        }
        grid_arrive(c, b0 + 0);
        // S2: self-attention and its output projection, x_cur += ...
        if (sched.unit) {
            grid_wait(c, b0 + 0);
            self_stage(c, p, la, sched, nr, x_cur);
        }
        grid_arrive(c, b0 + 1);
        // S3: cross-attention block, x_next = x_cur + ...
        if (sched.unit) {
            grid_wait(c, b0 + 1);
            cross_stage(c, p, la, sched, nr, x_cur, x_next);
        }
        grid_arrive(c, b0 + 2);
        // S4: FFN hidden layer raw; side jobs: LN3 statistics, clear [q | k | v] for the next layer
        grid_wait(c, b0 + 2);
        if (static_cast<int>(blockIdx.x) < n) row_stats(c, x_next, blockIdx.x, d, p.eps, p.stats3 + blockIdx.x);
        zero_floats(c, p.qkv, static_cast<size_t>(n) * 3 * d);
        {
            TileArgs a{};
            a.src = x_next; a.ld_src = d; a.gamma = la.ln3_g;
            a.out = p.hid; a.ldo = F; a.n_features = F; a.bias = nullptr;
            tile_stage<T_GAMMA>(c, sched.s4_begin, sched.s4_end, sched.kb_d, a, n);
        }
        grid_arrive(c, b0 + 3);
        // S5: x_next += relu(LN3-corrected hidden) W2^T + b2
        grid_wait(c, b0 + 3);
        {
            TileArgs a{};
            a.src = p.hid; a.ld_src = F; a.c1 = la.c1_ff; a.c2 = la.c2_ff; a.stats = p.stats3;
            a.out = x_next; a.ldo = d; a.n_features = d; a.bias = la.b_ff2;
            tile_stage<T_LN_RELU>(c, sched.s5_begin, sched.s5_end, sched.kb_f, a, n);
        }
        grid_arrive(c, b0 + 4);
    }
    if (c.tid == 0 && abort_flag) {
        atomicExch(c.bars + c.n_bars, 1);
        atomicExch(&p.state->error, kErrTimeout);
    }
}

}  // namespace mega
}  // namespace aed
