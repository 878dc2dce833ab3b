// Per-step kernels of the AED decoder: row bookkeeping, embedding, LayerNorm, CUDA-core GEMM with fused
// epilogues (fp32 mode and fallback shapes), flash-decoding attention over ragged caches, argmax finalisation.
#pragma once
#include "common.cuh"

namespace aed {

// ------------------------------------------------------------------------------------------------------------
// Row bookkeeping: compaction of the utterances that take part in the next step, in a fixed visiting order.
//   active_list[r] = utterance id of compact row r;  state->n_active = number of rows.
// An utterance takes part if it is not retired, the caller's mask (if any) selects it, and its self-attention
// cache still has room; a selected utterance with a full cache raises the sticky error instead of overflowing.
// ------------------------------------------------------------------------------------------------------------
// It also fills the row table: row_info[r] = (utterance, t_u, encoder length, encoder offset) for every compact
// row, and utterance -1 for the slots past the last row, so that a kernel needs one 16-byte load per row.
// The batch size is read from the decode state, not passed by value: a captured step graph outlives the batch it
// was recorded for and is replayed for later batches of other sizes.
__global__ void build_active_kernel(const uint8_t *__restrict__ mask, const int32_t *__restrict__ retired,
                                    const int32_t *__restrict__ t_u, int max_dec_len,
                                    int32_t *__restrict__ active_list, DecState *state,
                                    const int32_t *__restrict__ enc_len, const int32_t *__restrict__ enc_off,
                                    int4 *__restrict__ row_info, int row_slots, const int32_t *__restrict__ order)
{
    AED_TRACE_BEGIN(state, 1);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the next kernel may become resident; it waits for this one inside
    __shared__ int warp_counts[32];
    __shared__ int base;
    const int batch = state->batch;
    if (threadIdx.x == 0) base = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int start = 0; start < batch; start += blockDim.x) {
        // utterances are visited in the given order (longest encoder output first), so compact rows come out
        // sorted by encoder length: the attention blocks of the longest rows are scheduled first
        const int i = start + threadIdx.x;
        const int u = i < batch ? order[i] : batch;
        bool take = false;
        if (u < batch) {
            take = retired[u] == 0 && (mask == nullptr || mask[u] != 0);
            if (take && t_u[u] >= max_dec_len) { take = false; atomicExch(&state->error, 1); }
        }
        unsigned ballot = __ballot_sync(0xffffffffu, take);
        if (lane == 0) warp_counts[warp] = __popc(ballot);
        __syncthreads();
        int before = base;
        for (int w = 0; w < warp; ++w) before += warp_counts[w];
        if (take) {
            const int slot = before + __popc(ballot & ((1u << lane) - 1u));
            active_list[slot] = u;
            row_info[slot] = make_int4(u, t_u[u], enc_len[u], enc_off[u]);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int total = 0;
            for (int w = 0; w < n_warps; ++w) total += warp_counts[w];
            base += total;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { state->n_active = base; state->grid_sync = 0; }
    for (int r = base + threadIdx.x; r < row_slots; r += blockDim.x) row_info[r] = make_int4(-1, 0, 0, 0);
}

// Sinusoidal position table PE[t][2i] = sin(t / 10000^(2i/d)), PE[t][2i+1] = cos(same), evaluated in double.
__global__ void fill_pe_kernel(float *pe, int max_len, int d)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= max_len * d) return;
    int t = idx / d, i = idx % d;
    double angle = static_cast<double>(t) / pow(10000.0, (2.0 * (i / 2)) / static_cast<double>(d));
    pe[idx] = static_cast<float>((i & 1) ? cos(angle) : sin(angle));
}

// x[r] = E[token of utterance] * sqrt(d) + PE[t_u]
template <typename T>
__global__ void embed_kernel(const DecState *state, const int32_t *__restrict__ active_list,
                             const int32_t *__restrict__ tokens, const int32_t *__restrict__ t_u,
                             const T *__restrict__ embed, const float *__restrict__ pe, int d, int vocab, float scale,
                             float *__restrict__ x, float *__restrict__ zero_buf = nullptr, int zero_cols = 0,
                             float *__restrict__ zero_buf2 = nullptr, int zero_cols2 = 0)
{
    AED_TRACE_BEGIN(state, 2);
    // may be launched with programmatic stream serialization, right behind the row compaction
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int r = blockIdx.x;
    if (r >= state->n_active) return;
    int u = active_list[r];
    int tok = tokens[u];
    tok = min(max(tok, 0), vocab - 1);
    int t = t_u[u];
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        x[(size_t)r * d + i] = to_f32(embed[(size_t)tok * d + i]) * scale + pe[(size_t)t * d + i];
    for (int i = threadIdx.x; i < zero_cols; i += blockDim.x) zero_buf[(size_t)r * zero_cols + i] = 0.f;
    for (int i = threadIdx.x; i < zero_cols2; i += blockDim.x) zero_buf2[(size_t)r * zero_cols2 + i] = 0.f;
}

// out[r] = g * (x[r] - mean) / sqrt(var + eps) + b, biased variance, two passes over a row held in registers.
template <typename T, int kMaxPerThread>
__global__ void layernorm_kernel(const DecState *state, const float *__restrict__ x, const T *__restrict__ g,
                                 const T *__restrict__ b, int d, float eps, float *__restrict__ out)
{
    int r = blockIdx.x;
    if (r >= state->n_active) return;
    __shared__ float red[32];
    __shared__ float stat;
    float v[kMaxPerThread];
    const float *xr = x + (size_t)r * d;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        v[j] = (i < d) ? xr[i] : 0.f;
        s += v[j];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    s = warp_sum(s);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) { float tsum = 0.f; for (int w = 0; w < n_warps; ++w) tsum += red[w]; stat = tsum / d; }
    __syncthreads();
    float mean = stat;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        float c = (i < d) ? v[j] - mean : 0.f;
        q += c * c;
    }
    q = warp_sum(q);
    __syncthreads();
    if (lane == 0) red[warp] = q;
    __syncthreads();
    if (threadIdx.x == 0) { float tsum = 0.f; for (int w = 0; w < n_warps; ++w) tsum += red[w]; stat = rsqrtf(tsum / d + eps); }
    __syncthreads();
    float rstd = stat;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        if (i < d) out[(size_t)r * d + i] = to_f32(g[i]) * (v[j] - mean) * rstd + to_f32(b[i]);
    }
}

// ------------------------------------------------------------------------------------------------------------
// CUDA-core GEMM  out[r, o] = sum_k A[r, k] * W[o, k] + bias[o]  with fused epilogues.
// 64 rows x 32 output features per block, K in slices of 32 staged through shared memory, 4x4 per thread.
// ------------------------------------------------------------------------------------------------------------
enum Epilogue { EPI_STORE = 0, EPI_RELU = 1, EPI_RESID = 2, EPI_QKV = 3, EPI_LOGITS = 4, EPI_CROSSKV = 5 };

template <typename CT>
struct GemmEpilogueArgs {
    float *out;                 // STORE / RELU: [rows, ldo];  RESID: x [rows, ldo];  QKV: q [rows, d]
    int ldo;
    // QKV: self-attention cache of this layer [batch][2][H][max_dec_len][64]
    CT *self_cache;
    const int32_t *active_list;
    const int32_t *t_u;
    int max_dec_len, d_model, n_heads;
    // LOGITS
    float *logits_out;          // [batch, vocab] by utterance, or nullptr
    unsigned long long *keys;   // [rows] packed argmax keys
    // CROSSKV: store of this layer [2][H][frame_capacity][64]
    CT *cross_store;
    int frame_capacity;
    int frame0;                 // CROSSKV: store row of the first frame (an utterance admitted into a slot of its own)
};

template <typename AT, typename WT, typename CT, int EPI>
__global__ void __launch_bounds__(128)
gemm_rows_kernel(const DecState *state, int rows_fixed, const AT *__restrict__ A, int lda,
                 const WT *__restrict__ W, const WT *__restrict__ bias, int M, int K, GemmEpilogueArgs<CT> ep)
{
    constexpr int BM = 64, BN = 32, BK = 32;
    const int n_rows = (rows_fixed >= 0) ? rows_fixed : state->n_active;
    const int row0 = blockIdx.y * BM, o0 = blockIdx.x * BN;
    if (row0 >= n_rows) return;
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Ws[BK][BN + 4];
    const int tid = threadIdx.x, tx = tid & 7, ty = tid >> 3;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += BK) {
        // A tile: 64 rows x 32 k, 4 elements per load
        for (int idx = tid; idx < BM * BK / 4; idx += 128) {
            int r = idx / (BK / 4), kq = (idx % (BK / 4)) * 4;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (row0 + r < n_rows) load4(A + (size_t)(row0 + r) * lda + k0 + kq, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) As[kq + j][r] = v[j];
        }
        for (int idx = tid; idx < BN * BK / 4; idx += 128) {
            int o = idx / (BK / 4), kq = (idx % (BK / 4)) * 4;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (o0 + o < M) load4(W + (size_t)(o0 + o) * K + k0 + kq, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) Ws[kq + j][o] = v[j];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float4 a4 = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
            float4 w4 = *reinterpret_cast<const float4 *>(&Ws[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }

    // epilogue
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = row0 + ty * 4 + i;
        const bool row_ok = r < n_rows;
        float best = -INFINITY;
        uint32_t best_idx = 0;
        int u = 0, t = 0;
        if (row_ok && (EPI == EPI_QKV || EPI == EPI_LOGITS)) u = ep.active_list[r];
        if (row_ok && EPI == EPI_QKV) t = ep.t_u[u];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = o0 + tx * 4 + j;
            if (!row_ok || o >= M) continue;
            float v = acc[i][j] + (bias ? to_f32(bias[o]) : 0.f);
            if (EPI == EPI_STORE) {
                ep.out[(size_t)r * ep.ldo + o] = v;
            } else if (EPI == EPI_RELU) {
                ep.out[(size_t)r * ep.ldo + o] = fmaxf(v, 0.f);
            } else if (EPI == EPI_RESID) {
                ep.out[(size_t)r * ep.ldo + o] += v;
            } else if (EPI == EPI_QKV) {
                const int d = ep.d_model;
                if (o < d) {
                    ep.out[(size_t)r * d + o] = v;
                } else {
                    const int kv = (o - d) / d, c = (o - d) % d, h = c / kHeadDim, e = c % kHeadDim;
                    size_t off = ((((size_t)u * 2 + kv) * ep.n_heads + h) * ep.max_dec_len + t) * kHeadDim + e;
                    ep.self_cache[off] = from_f32<CT>(v);
                }
            } else if (EPI == EPI_LOGITS) {
                if (ep.logits_out) ep.logits_out[(size_t)u * M + o] = v;
                if (v > best) { best = v; best_idx = o; }
            } else if (EPI == EPI_CROSSKV) {
                const int d = ep.d_model;
                const int kv = o / d, c = o % d, h = c / kHeadDim, e = c % kHeadDim;
                size_t off = (((size_t)kv * ep.n_heads + h) * ep.frame_capacity + ep.frame0 + r) * kHeadDim + e;
                ep.cross_store[off] = from_f32<CT>(v);
            }
        }
        if (EPI == EPI_LOGITS) {
            // the 8 threads that share this row sit in consecutive lanes: reduce, then one atomic per block row
            unsigned long long key = (row_ok && best > -INFINITY) ? argmax_key(best, best_idx) : 0ull;
#pragma unroll
            for (int off = 1; off < 8; off <<= 1) {
                unsigned long long other = __shfl_xor_sync(0xffffffffu, key, off);
                key = other > key ? other : key;
            }
            if (tx == 0 && row_ok && key != 0ull) atomicMax(ep.keys + r, key);
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// Flash-decoding attention over ragged caches.  One warp per (row, head, chunk of 64 positions): lanes are
// 4 position groups x 8 dimension groups, each lane holds 8 of the 64 head dimensions (one 128-bit load of a
// bf16 key or value row segment).  Scores are reduced over the 8 dimension lanes with shuffles, softmax is
// kept online per position group and merged over the 4 groups at the end.  Each work item writes
// (running max, running sum, 64 un-normalised accumulators); the combine kernel merges the chunks of a row.
//   SELF : keys/values of utterance u, head h at  cache[((u*2 + kv)*H + h)*max_len*64],  length t_u + 1
//   CROSS: keys/values at store[(kv*H + h)*capacity*64 + enc_off[u]*64],                 length enc_len[u]
// ------------------------------------------------------------------------------------------------------------
// With kAppend (self-attention after a split-K projection) q, k and v of the new position sit side by side in
// one fp32 row [q | k | v] of `q`; the warp whose chunk holds position t_u first stores k and v into the cache.
template <typename CT, bool kCross, bool kAppend = false>
__global__ void __launch_bounds__(128)
attn_partial_kernel(const DecState *state, const int32_t *__restrict__ active_list, const float *__restrict__ q,
                    int ldq, CT *__restrict__ cache, int n_heads, int seq_capacity,
                    const int32_t *__restrict__ t_u, const int32_t *__restrict__ enc_off,
                    const int32_t *__restrict__ enc_len, int max_chunks, float scale, float *__restrict__ partials)
{
    const int rh = blockIdx.x;
    const int r = rh / n_heads, h = rh % n_heads;
    if (r >= state->n_active) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.y * 4 + warp;
    const int u = active_list[r];
    const int len = kCross ? enc_len[u] : t_u[u] + 1;
    const int p0 = chunk * kAttnChunk;
    if (chunk >= max_chunks || p0 >= len) return;
    const int p1 = min(len, p0 + kAttnChunk);
    const CT *kbase, *vbase;
    if (kCross) {
        kbase = cache + ((size_t)(0 * n_heads + h) * seq_capacity + enc_off[u]) * kHeadDim;
        vbase = cache + ((size_t)(1 * n_heads + h) * seq_capacity + enc_off[u]) * kHeadDim;
    } else {
        kbase = cache + (((size_t)u * 2 + 0) * n_heads + h) * (size_t)seq_capacity * kHeadDim;
        vbase = cache + (((size_t)u * 2 + 1) * n_heads + h) * (size_t)seq_capacity * kHeadDim;
    }
    const int dg = lane & 7, pg = lane >> 3;
    if (kAppend && !kCross && len - 1 >= p0 && len - 1 < p1) {
        if (lane < 16) {
            const int kv = lane >> 3, d_model = n_heads * kHeadDim;
            float nv[8];
            load8(q + (size_t)r * ldq + (1 + kv) * d_model + h * kHeadDim + dg * 8, nv);
            CT *dst = const_cast<CT *>(kv ? vbase : kbase) + (size_t)(len - 1) * kHeadDim + dg * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = from_f32<CT>(nv[i]);
        }
        __syncwarp();
    }
    float qv[8];
    load8(q + (size_t)r * ldq + h * kHeadDim + dg * 8, qv);
#pragma unroll
    for (int i = 0; i < 8; ++i) qv[i] *= scale;

    float m = -INFINITY, l = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    for (int p = p0 + pg; p < p0 + kAttnChunk; p += 4) {   // uniform trip count: shuffles need all lanes
        const bool ok = p < p1;
        float kv[8], s = 0.f;
        if (ok) {
            load8(kbase + (size_t)p * kHeadDim + dg * 8, kv);
#pragma unroll
            for (int i = 0; i < 8; ++i) s = fmaf(qv[i], kv[i], s);
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        if (ok) {
            float vv[8];
            load8(vbase + (size_t)p * kHeadDim + dg * 8, vv);
            float m_new = fmaxf(m, s);
            float corr = expf(m - m_new), pr = expf(s - m_new);
            l = l * corr + pr;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(pr, vv[i], acc[i] * corr);
            m = m_new;
        }
    }
    // merge the 4 position groups (lanes differing in bits 3 and 4)
#pragma unroll
    for (int off = 8; off < 32; off <<= 1) {
        float m_o = __shfl_xor_sync(0xffffffffu, m, off);
        float l_o = __shfl_xor_sync(0xffffffffu, l, off);
        float m_new = fmaxf(m, m_o);
        float c_self = (m == -INFINITY) ? 0.f : expf(m - m_new);
        float c_oth = (m_o == -INFINITY) ? 0.f : expf(m_o - m_new);
        l = l * c_self + l_o * c_oth;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float a_o = __shfl_xor_sync(0xffffffffu, acc[i], off);
            acc[i] = acc[i] * c_self + a_o * c_oth;
        }
        m = m_new;
    }
    float *dst = partials + ((size_t)rh * max_chunks + chunk) * kPartialStride;
    if (lane == 0) { dst[0] = m; dst[1] = l; }
    if (pg == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[2 + dg * 8 + i] = acc[i];
    }
}


// ------------------------------------------------------------------------------------------------------------
// Single-pass attention for one (row, head) per block: no scratch, no second kernel.  Warp w takes the
// 16-position chunks w, w + n_warps, ...; within a chunk every lane issues its 4 key and 4 value loads (128 bits
// each) together, so one memory latency covers the chunk, then reduces the scores with shuffles.
// Warps keep a running (max, sum, accumulator) and are merged through shared memory at the end.
// Lanes: 8 dimension groups (8 head dimensions each) x 4 position groups.
//   kAppend (self-attention): q row is [q | k | v]; k and v of the new position are stored first.
//   Output: fp32 [row, d] (out) and/or bf16 high/low planes (out_hi/out_lo), whichever pointers are non-null.
// ------------------------------------------------------------------------------------------------------------
template <typename CT> struct RawLane;
template <> struct RawLane<__nv_bfloat16> {
    uint4 v;
    __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = *reinterpret_cast<const uint4 *>(p); }
    __device__ __forceinline__ void zero() { v = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void set(const float (&f)[8])          // rounds to bf16, as the cache stores it
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 pr = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&pr);
        }
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __device__ __forceinline__ void store(__nv_bfloat16 *p) const { *reinterpret_cast<uint4 *>(p) = v; }
    __device__ __forceinline__ void get(float (&f)[8]) const
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
    }
};
template <> struct RawLane<fp8e4m3> {
    uint2 v;                                                                   // 8 bytes = 8 values
    __device__ __forceinline__ void load(const fp8e4m3 *p) { v = *reinterpret_cast<const uint2 *>(p); }
    __device__ __forceinline__ void zero() { v = make_uint2(0u, 0u); }
    __device__ __forceinline__ void set(const float (&f)[8])
    {
        v.x = static_cast<uint32_t>(pack_e4m3x2(f[0], f[1])) | (static_cast<uint32_t>(pack_e4m3x2(f[2], f[3])) << 16);
        v.y = static_cast<uint32_t>(pack_e4m3x2(f[4], f[5])) | (static_cast<uint32_t>(pack_e4m3x2(f[6], f[7])) << 16);
    }
    __device__ __forceinline__ void store(fp8e4m3 *p) const { *reinterpret_cast<uint2 *>(p) = v; }
    __device__ __forceinline__ void get(float (&f)[8]) const
    {
        const float2 a = unpack_e4m3x2(static_cast<uint16_t>(v.x & 0xFFFFu)), b = unpack_e4m3x2(static_cast<uint16_t>(v.x >> 16));
        const float2 c = unpack_e4m3x2(static_cast<uint16_t>(v.y & 0xFFFFu)), d = unpack_e4m3x2(static_cast<uint16_t>(v.y >> 16));
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
    }
};
template <> struct RawLane<float> {
    float4 a, b;
    __device__ __forceinline__ void load(const float *p) { a = *reinterpret_cast<const float4 *>(p); b = *reinterpret_cast<const float4 *>(p + 4); }
    __device__ __forceinline__ void zero() { a = make_float4(0.f, 0.f, 0.f, 0.f); b = a; }
    __device__ __forceinline__ void set(const float (&f)[8]) { a = make_float4(f[0], f[1], f[2], f[3]); b = make_float4(f[4], f[5], f[6], f[7]); }
    __device__ __forceinline__ void store(float *p) const { *reinterpret_cast<float4 *>(p) = a; *reinterpret_cast<float4 *>(p + 4) = b; }
    __device__ __forceinline__ void get(float (&f)[8]) const
    { f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w; }
};

// Head dimensions per lane.  8 for every storage type: with single-byte keys and values, 16 per lane (one 16-byte load
// per row and lane, 32 positions per warp and pass) was measured slower at 512 rows (693 against 654 ms per pass of
// the 24-layer batch-512 workload): the kernel is bound by how many loads its resident warps keep in flight, not by
// bytes per load, and the wider lanes cost a resident block per SM.
template <typename CT> struct LaneWidth { static constexpr int kE = 8; };
// positions per warp and iteration: 4 passes over the 32 / (64 / kE) position groups of a warp
template <typename CT> constexpr int fused_chunk() { return 4 * (32 / (kHeadDim / LaneWidth<CT>::kE)); }
constexpr int kFusedMaxWarps = 8;

// 2^x by the hardware approximation (relative error about 2^-22): softmax weights of the single-pass attention kernel
__device__ __forceinline__ float exp2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int N> __device__ __forceinline__ void load_n(const float *p, float (&v)[N])
{
#pragma unroll
    for (int i = 0; i < N; i += 4) {
        const float4 a = *reinterpret_cast<const float4 *>(p + i);
        v[i] = a.x; v[i + 1] = a.y; v[i + 2] = a.z; v[i + 3] = a.w;
    }
}

// kPipe: the loads of a warp's next chunk are issued before the current chunk is reduced (twice the K/V registers,
// so only two blocks per SM: for grids that fit anyway).
// kRowStats: the block computes (mean, rstd) of its row of stats_x itself instead of reading ln_stats.
template <typename CT, bool kCross, bool kAppend, bool kPipe = false, bool kRowStats = false>
__global__ void __launch_bounds__(kFusedMaxWarps * 32, ((kAppend || kPipe) ? 2 : (LaneWidth<CT>::kE > 8 ? 3 : 4)))      // self-attention holds the new key/value as well; wider lanes need more registers
attn_fused_kernel(const DecState *state, const int4 *__restrict__ row_info, const float *__restrict__ q, int ldq,
                  CT *__restrict__ cache, int n_heads, int seq_capacity, float scale,
                  float *__restrict__ out, __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo, int ldo,
                  const float2 *__restrict__ ln_stats, const float *__restrict__ ln_c1, const float *__restrict__ ln_c2,
                  const float *__restrict__ stats_x = nullptr, float ln_eps = 0.f)
{
    // stats_x: rows [*, heads * 64] whose (mean, rstd) this block computes itself instead of reading ln_stats (the
    // kernel before this one completed those rows, so nobody could have computed the statistics earlier).
    // Launched with programmatic stream serialization.  Before the dependency wait only data that no kernel of
    // this step writes is touched: the row table (written by the step's first kernel, which ran to completion
    // before any programmatic launch of the step) and, for cross-attention, the encoder K/V store.
    __shared__ float sm_m[kFusedMaxWarps], sm_l[kFusedMaxWarps];
    __shared__ float sm_acc[kFusedMaxWarps][kHeadDim];
    __shared__ float2 sm_red[kFusedMaxWarps];
    const int rh = blockIdx.x;
    const int r = rh / n_heads, h = rh % n_heads;
    const int4 ri = row_info[r];                       // (utterance, t_u, encoder length, encoder offset)
    if (ri.x < 0) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    const int u = ri.x;
    const int len = kCross ? ri.z : ri.y + 1;
    const CT *kbase, *vbase;
    if (kCross) {
        kbase = cache + ((size_t)(0 * n_heads + h) * seq_capacity + ri.w) * kHeadDim;
        vbase = cache + ((size_t)(1 * n_heads + h) * seq_capacity + ri.w) * kHeadDim;
    } else {
        kbase = cache + (((size_t)u * 2 + 0) * n_heads + h) * (size_t)seq_capacity * kHeadDim;
        vbase = cache + (((size_t)u * 2 + 1) * n_heads + h) * (size_t)seq_capacity * kHeadDim;
    }
    // Positions that earlier steps (or the precompute) wrote are static for this kernel; the position appended
    // by this step (self-attention only) is taken from the projection output after the dependency wait.
    const int len_static = (kAppend && !kCross) ? len - 1 : len;
    constexpr int kE = LaneWidth<CT>::kE, kDG = kHeadDim / kE, kPG = 32 / kDG, kChunk = 4 * kPG;
    const int dg = lane % kDG, pg = lane / kDG;      // lanes: kDG groups of kE head dimensions x kPG positions
    RawLane<CT> rk[4], rv[4];
    // Self-attention without an append of its own (prefill pass): the cache positions it reads are written by the
    // kernel before it, so nothing is loaded ahead of the dependency wait.
    if (!kCross && !kAppend) asm volatile("griddepcontrol.wait;" ::: "memory");
    {
        // This warp's first chunk starts streaming while the kernel that produces the query is still running.
        const int p0 = warp * kChunk;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = p0 + i * kPG + pg;
            if (p < len_static) {
                rk[i].load(kbase + (size_t)p * kHeadDim + dg * kE);
                rv[i].load(vbase + (size_t)p * kHeadDim + dg * kE);
            } else { rk[i].zero(); rv[i].zero(); }
        }
        // later chunks of this warp: pull them into L2 now (one 128-byte row per lane group)
        if (dg == 0) {
            for (int q0 = p0 + n_warps * kChunk; q0 < len_static; q0 += n_warps * kChunk) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int p = q0 + i * kPG + pg;
                    if (p < len_static) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(kbase + (size_t)p * kHeadDim));
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(vbase + (size_t)p * kHeadDim));
                    }
                }
            }
        }
    }
    // The LayerNorm-fold constants of this block's columns are static as well (read once per step and layer, so
    // they come from DRAM): requested here, before the dependency wait.
    const int new_chunk = (len - 1) / kChunk;
    const bool owns_new = kAppend && !kCross && warp == new_chunk % n_warps;
    const int d_model = n_heads * kHeadDim;
    const int qcol = h * kHeadDim + dg * kE;
    float qc1[kE], qc2[kE], kc1[kE], kc2[kE], vc1[kE], vc2[kE];
    const bool fold = ln_stats != nullptr || kRowStats;
    if (fold) {
        load_n<kE>(ln_c1 + qcol, qc1); load_n<kE>(ln_c2 + qcol, qc2);
        if (owns_new) {
            load_n<kE>(ln_c1 + d_model + qcol, kc1); load_n<kE>(ln_c2 + d_model + qcol, kc2);
            load_n<kE>(ln_c1 + 2 * d_model + qcol, vc1); load_n<kE>(ln_c2 + 2 * d_model + qcol, vc2);
        }
    }
    AED_TRACE_RESERVE(tcur, state, (threadIdx.x == 0 && blockIdx.x == 0) ? 6u : 0u);
    AED_TRACE_PUT_NS(state, tcur, 8 + (kCross ? 1 : 0));      // resident, first chunk requested
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    AED_TRACE_PUT(state, tcur, 3);                          // dependency resolved
    // Everything this block needs from earlier kernels is requested in one round: statistics, query, and (in the
    // warp that owns the new position) the new key and value.  When the projection ran on gamma*x, its raw output
    // y becomes rstd*(y - mean*c1) + c2 here.
    float2 st = make_float2(0.f, 1.f);
    float qv[kE], kn[kE], vn[kE];
    if (ln_stats) st = ln_stats[r];
    load_n<kE>(q + (size_t)r * ldq + qcol, qv);
    if (owns_new) {
        load_n<kE>(q + (size_t)r * ldq + d_model + qcol, kn);
        load_n<kE>(q + (size_t)r * ldq + 2 * d_model + qcol, vn);
    }
    if (kRowStats) {
        // mean and rstd of row r in one pass over deviations from the row's first element (a row whose mean is far
        // from zero loses nothing to cancellation that way): var = (S2 - S1^2 / n) / n, mean = x0 + S1 / n
        const float *xr = stats_x + (size_t)r * d_model;
        const float x0 = xr[0];
        float s1 = 0.f, s2 = 0.f;
        for (int idx = threadIdx.x * 4; idx < d_model; idx += blockDim.x * 4) {
            const float4 v = *reinterpret_cast<const float4 *>(xr + idx);
            const float d0 = v.x - x0, d1 = v.y - x0, d2 = v.z - x0, d3 = v.w - x0;
            s1 += (d0 + d1) + (d2 + d3);
            s2 += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
        }
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        if (lane == 0) sm_red[warp] = make_float2(s1, s2);
        __syncthreads();
        float t1 = 0.f, t2 = 0.f;
        for (int w = 0; w < n_warps; ++w) { t1 += sm_red[w].x; t2 += sm_red[w].y; }
        const float inv_n = 1.f / d_model;
        const float var = fmaxf((t2 - t1 * t1 * inv_n) * inv_n, 0.f);
        st = make_float2(x0 + t1 * inv_n, rsqrtf(var + ln_eps));
    }
    if (fold) {
#pragma unroll
        for (int i = 0; i < kE; ++i) qv[i] = fmaf(st.y, qv[i] - st.x * qc1[i], qc2[i]);
    }
#pragma unroll
    for (int i = 0; i < kE; ++i) qv[i] *= scale * 1.4426950408889634f;      // scores in units of ln 2: exponentials below are 2^x
    RawLane<CT> new_k, new_v;
    if (owns_new) {
        if (fold) {
#pragma unroll
            for (int i = 0; i < kE; ++i) {
                kn[i] = fmaf(st.y, kn[i] - st.x * kc1[i], kc2[i]);
                vn[i] = fmaf(st.y, vn[i] - st.x * vc1[i], vc2[i]);
            }
        }
        new_k.set(kn);
        new_v.set(vn);
        if (pg == 0) {      // append to the cache; no other block reads this position during the kernel
            new_k.store(const_cast<CT *>(kbase) + (size_t)(len - 1) * kHeadDim + dg * kE);
            new_v.store(const_cast<CT *>(vbase) + (size_t)(len - 1) * kHeadDim + dg * kE);
        }
    }

    AED_TRACE_PUT(state, tcur, 4);                          // query ready (statistics, fold)
    float m = -INFINITY, l = 0.f, acc[kE];
#pragma unroll
    for (int i = 0; i < kE; ++i) acc[i] = 0.f;
    bool loaded = true;
    RawLane<CT> nk[4], nv[4];
    for (int p0 = warp * kChunk; p0 < len; p0 += n_warps * kChunk) {
        if (kPipe) {
            const int pn = p0 + n_warps * kChunk;
            if (pn < len) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int p = pn + i * kPG + pg;
                    if (p < len_static) {
                        nk[i].load(kbase + (size_t)p * kHeadDim + dg * kE);
                        nv[i].load(vbase + (size_t)p * kHeadDim + dg * kE);
                    } else { nk[i].zero(); nv[i].zero(); }
                }
            }
        } else if (!loaded) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {          // keys and values of the chunk are requested together
                const int p = p0 + i * kPG + pg;
                if (p < len_static) {
                    rk[i].load(kbase + (size_t)p * kHeadDim + dg * kE);
                    rv[i].load(vbase + (size_t)p * kHeadDim + dg * kE);
                } else { rk[i].zero(); rv[i].zero(); }
            }
        }
        loaded = false;
        if (owns_new && p0 == new_chunk * kChunk) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (p0 + i * kPG + pg == len - 1) { rk[i] = new_k; rv[i] = new_v; }
        }
        float s[4], cmax = -INFINITY;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float kf[kE], d = 0.f;
            rk[i].get(kf);
#pragma unroll
            for (int j = 0; j < kE; ++j) d = fmaf(qv[j], kf[j], d);
#pragma unroll
            for (int o = 1; o < kDG; o <<= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            s[i] = (p0 + i * kPG + pg < len) ? d : -INFINITY;
            cmax = fmaxf(cmax, s[i]);
        }
#pragma unroll
        for (int o = kDG; o < 32; o <<= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));     // chunk max, uniform over the warp, finite
        const float m_new = fmaxf(m, cmax);
        const float corr = exp2_fast(m - m_new);
        l *= corr;
#pragma unroll
        for (int j = 0; j < kE; ++j) acc[j] *= corr;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float pr = exp2_fast(s[i] - m_new);      // 2^(-inf) = 0 for positions past the end
            float vf[kE];
            rv[i].get(vf);
            l += pr;
#pragma unroll
            for (int j = 0; j < kE; ++j) acc[j] = fmaf(pr, vf[j], acc[j]);
        }
        m = m_new;
        if (kPipe) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { rk[i] = nk[i]; rv[i] = nv[i]; }
        }
    }
    AED_TRACE_PUT(state, tcur, 5);                          // all chunks of this warp reduced
    // sum the position groups (they share m)
#pragma unroll
    for (int o = kDG; o < 32; o <<= 1) {
        l += __shfl_xor_sync(0xffffffffu, l, o);
#pragma unroll
        for (int j = 0; j < kE; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    }
    if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    if (pg == 0) {
#pragma unroll
        for (int j = 0; j < kE; ++j) sm_acc[warp][dg * kE + j] = acc[j];
    }
    __syncthreads();
    if (threadIdx.x < kHeadDim) {
        float big = -INFINITY;
        for (int w = 0; w < n_warps; ++w) big = fmaxf(big, sm_m[w]);
        float lsum = 0.f, a = 0.f;
        for (int w = 0; w < n_warps; ++w) {
            const float wgt = (sm_m[w] == -INFINITY) ? 0.f : exp2_fast(sm_m[w] - big);
            lsum = fmaf(sm_l[w], wgt, lsum);
            a = fmaf(sm_acc[w][threadIdx.x], wgt, a);
        }
        const float o = a / lsum;
        const size_t off = (size_t)r * ldo + h * kHeadDim + threadIdx.x;
        if (out) out[off] = o;
        if (out_hi) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(o);
            out_hi[off] = hi;
            out_lo[off] = __float2bfloat16_rn(o - __bfloat162float(hi));
        }
    }
    AED_TRACE_PUT_NS(state, tcur, 7);                       // output written
}

// Merge the chunk partials of each (row, head): one warp per pair, 2 head dimensions per lane.
template <bool kCross>
__global__ void __launch_bounds__(128)
attn_combine_kernel(const DecState *state, const int32_t *__restrict__ active_list, const float *__restrict__ partials,
                    int n_heads, const int32_t *__restrict__ t_u, const int32_t *__restrict__ enc_len, int max_chunks,
                    float *__restrict__ out, int ldo)
{
    const int rh = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int r = rh / n_heads, h = rh % n_heads;
    if (r >= state->n_active) return;
    const int u = active_list[r];
    const int len = kCross ? enc_len[u] : t_u[u] + 1;
    const int n_chunks = (len + kAttnChunk - 1) / kAttnChunk;
    const float *src = partials + (size_t)rh * max_chunks * kPartialStride;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, src[(size_t)c * kPartialStride]);
    float l = 0.f, a0 = 0.f, a1 = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float *p = src + (size_t)c * kPartialStride;
        float w = expf(p[0] - m);
        l = fmaf(p[1], w, l);
        a0 = fmaf(p[2 + lane * 2], w, a0);
        a1 = fmaf(p[3 + lane * 2], w, a1);
    }
    float inv = 1.f / l;
    float2 o = make_float2(a0 * inv, a1 * inv);
    *reinterpret_cast<float2 *>(out + (size_t)r * ldo + h * kHeadDim + lane * 2) = o;
}

// LayerNorm whose result is written as bf16 high and low planes [row, d]; the same block also clears the fp32
// rows that the following split-K projection accumulates into (zero_cols columns of zero_buf, if any).
template <int kMaxPerThread>
__global__ void layernorm_planes_kernel(const DecState *state, const float *__restrict__ x,
                                        const __nv_bfloat16 *__restrict__ g, const __nv_bfloat16 *__restrict__ b, int d,
                                        float eps, __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo,
                                        float *__restrict__ zero_buf, int zero_cols)
{
    AED_TRACE_BEGIN(state, 4);
    // launched with programmatic stream serialization: nothing of the previous kernel is touched before this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int r = blockIdx.x;
    if (r >= state->n_active) return;
    __shared__ float red[32];
    __shared__ float stat;
    float v[kMaxPerThread];
    const float *xr = x + (size_t)r * d;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        v[j] = (i < d) ? xr[i] : 0.f;
        s += v[j];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    s = warp_sum(s);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) { float tsum = 0.f; for (int w = 0; w < n_warps; ++w) tsum += red[w]; stat = tsum / d; }
    __syncthreads();
    const float mean = stat;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        float c = (i < d) ? v[j] - mean : 0.f;
        q += c * c;
    }
    q = warp_sum(q);
    __syncthreads();
    if (lane == 0) red[warp] = q;
    __syncthreads();
    if (threadIdx.x == 0) { float tsum = 0.f; for (int w = 0; w < n_warps; ++w) tsum += red[w]; stat = rsqrtf(tsum / d + eps); }
    __syncthreads();
    const float rstd = stat;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        int i = threadIdx.x + j * blockDim.x;
        if (i < d) {
            const float y = to_f32(g[i]) * (v[j] - mean) * rstd + to_f32(b[i]);
            const __nv_bfloat16 hi = __float2bfloat16_rn(y);
            out_hi[(size_t)r * d + i] = hi;
            out_lo[(size_t)r * d + i] = __float2bfloat16_rn(y - __bfloat162float(hi));
        }
    }
    for (int i = threadIdx.x; i < zero_cols; i += blockDim.x) zero_buf[(size_t)r * zero_cols + i] = 0.f;
}

// ------------------------------------------------------------------------------------------------------------
// Activation planes for steps with many rows.  There the projections fetch their activation operand ready-made
// (bf16 high plane + bf16 low plane = value - high) instead of converting it in every feature tile.
// Both kernels start with a programmatic-dependency wait and may be launched ahead of their predecessor's end.
// ------------------------------------------------------------------------------------------------------------
// planes of gamma * x, the LayerNorm statistics (mean, rstd) of every row, and the clearing of the fp32 rows a later
// split-K projection accumulates into (zero_cols columns of zero_buf, if any).  One block per row.
template <int kMaxPerThread>
__global__ void gamma_planes_kernel(const DecState *state, const float *__restrict__ x, const __nv_bfloat16 *__restrict__ g,
                                    int d, float eps, float2 *__restrict__ stats_out, __nv_bfloat16 *__restrict__ out_hi,
                                    __nv_bfloat16 *__restrict__ out_lo, float *__restrict__ zero_buf, int zero_cols)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x;
    if (r >= state->n_active) return;
    __shared__ float red[32];
    __shared__ float stat;
    float v[kMaxPerThread];
    const float *xr = x + (size_t)r * d;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        const int i = threadIdx.x + j * blockDim.x;
        v[j] = (i < d) ? xr[i] : 0.f;
        s += v[j];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    s = warp_sum(s);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) { float t = 0.f; for (int w = 0; w < n_warps; ++w) t += red[w]; stat = t / d; }
    __syncthreads();
    const float mean = stat;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        const int i = threadIdx.x + j * blockDim.x;
        const float c = (i < d) ? v[j] - mean : 0.f;
        q += c * c;
    }
    q = warp_sum(q);
    __syncthreads();
    if (lane == 0) red[warp] = q;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < n_warps; ++w) t += red[w];
        stats_out[r] = make_float2(mean, rsqrtf(t / d + eps));
    }
#pragma unroll
    for (int j = 0; j < kMaxPerThread; ++j) {
        const int i = threadIdx.x + j * blockDim.x;
        if (i < d) {
            const float y = to_f32(g[i]) * v[j];
            const __nv_bfloat16 hi = __float2bfloat16_rn(y);
            out_hi[(size_t)r * d + i] = hi;
            out_lo[(size_t)r * d + i] = __float2bfloat16_rn(y - __bfloat162float(hi));
        }
    }
    for (int i = threadIdx.x; i < zero_cols; i += blockDim.x) zero_buf[(size_t)r * zero_cols + i] = 0.f;
}

// planes of relu(rstd * (hidden_raw - mean * c1) + c2): the FFN hidden layer after the folded first projection.
// grid: x = blocks of 1024 hidden features, y = rows.
__global__ void lnrelu_planes_kernel(const DecState *state, const float *__restrict__ hid, int f,
                                     const float2 *__restrict__ stats, const float *__restrict__ c1,
                                     const float *__restrict__ c2, __nv_bfloat16 *__restrict__ out_hi,
                                     __nv_bfloat16 *__restrict__ out_lo)
{
    const int r = blockIdx.y;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (i < f) {                       // static operands before the dependency wait
        a = *reinterpret_cast<const float4 *>(c1 + i);
        b = *reinterpret_cast<const float4 *>(c2 + i);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (r >= state->n_active || i >= f) return;
    const float2 st = stats[r];
    const float4 h = *reinterpret_cast<const float4 *>(hid + (size_t)r * f + i);
    const float y[4] = {fmaxf(fmaf(st.y, h.x - st.x * a.x, b.x), 0.f), fmaxf(fmaf(st.y, h.y - st.x * a.y, b.y), 0.f),
                        fmaxf(fmaf(st.y, h.z - st.x * a.z, b.z), 0.f), fmaxf(fmaf(st.y, h.w - st.x * a.w, b.w), 0.f)};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        hi[j] = __float2bfloat16_rn(y[j]);
        lo[j] = __float2bfloat16_rn(y[j] - __bfloat162float(hi[j]));
    }
    __nv_bfloat162 *ph = reinterpret_cast<__nv_bfloat162 *>(out_hi + (size_t)r * f + i);
    __nv_bfloat162 *pl = reinterpret_cast<__nv_bfloat162 *>(out_lo + (size_t)r * f + i);
    ph[0] = __halves2bfloat162(hi[0], hi[1]); ph[1] = __halves2bfloat162(hi[2], hi[3]);
    pl[0] = __halves2bfloat162(lo[0], lo[1]); pl[1] = __halves2bfloat162(lo[2], lo[3]);
}

// ------------------------------------------------------------------------------------------------------------
// Prompt prefill: several positions of every utterance in one pass.  A compact row is an (utterance, position)
// pair; a chunk covers `chunk` consecutive positions of every utterance of the batch.  Rows are ordered position
// major with the chunk's last position first (row = (chunk - 1 - j) * batch + i), so that the rows of the last
// position, the only ones whose logits matter, are rows 0 .. batch - 1.
// ------------------------------------------------------------------------------------------------------------
__global__ void build_prefill_rows_kernel(DecState *state, int chunk, int j0, int prompt_len, const int32_t *__restrict__ prompt,
                                          const int32_t *__restrict__ t_u, const int32_t *__restrict__ enc_len,
                                          const int32_t *__restrict__ enc_off, const int32_t *__restrict__ order,
                                          int32_t *__restrict__ active_list, int4 *__restrict__ row_info,
                                          int32_t *__restrict__ row_tok, int row_slots)
{
    const int batch = state->batch, rows = batch * chunk;
    for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < row_slots; r += gridDim.x * blockDim.x) {
        if (r < rows) {
            const int u = order[r % batch], j = chunk - 1 - r / batch;
            active_list[r] = u;
            row_info[r] = make_int4(u, t_u[u] + j, enc_len[u], enc_off[u]);
            row_tok[r] = prompt[(size_t)u * prompt_len + j0 + j];
        } else {
            row_info[r] = make_int4(-1, 0, 0, 0);
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { state->n_active = rows; state->grid_sync = 0; }
}

// x[r] = E[token of the row] * sqrt(d) + PE[position of the row]
template <typename T>
__global__ void embed_rows_kernel(const DecState *state, const int4 *__restrict__ row_info, const int32_t *__restrict__ row_tok,
                                  const T *__restrict__ embed, const float *__restrict__ pe, int d, int vocab, float scale,
                                  float *__restrict__ x, float *__restrict__ zero_buf, int zero_cols,
                                  float *__restrict__ zero_buf2 = nullptr, int zero_cols2 = 0)
{
    const int r = blockIdx.x;
    if (r >= state->n_active) return;
    const int tok = min(max(row_tok[r], 0), vocab - 1), t = row_info[r].y;
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        x[(size_t)r * d + i] = to_f32(embed[(size_t)tok * d + i]) * scale + pe[(size_t)t * d + i];
    for (int i = threadIdx.x; i < zero_cols; i += blockDim.x) zero_buf[(size_t)r * zero_cols + i] = 0.f;
    for (int i = threadIdx.x; i < zero_cols2; i += blockDim.x) zero_buf2[(size_t)r * zero_cols2 + i] = 0.f;
}

// Keys and values of every row into the self-attention cache (raw projection output with the LayerNorm fold applied,
// rounded as the cache stores it), before any row attends: in a prefill pass a row reads positions that other rows of
// the same pass append.  grid: (rows, heads), 64 threads.
template <typename CT>
__global__ void append_kv_kernel(const DecState *state, const int4 *__restrict__ row_info, const float *__restrict__ qkv, int ldq,
                                 CT *__restrict__ cache, int n_heads, int seq_capacity, const float2 *__restrict__ ln_stats,
                                 const float *__restrict__ ln_c1, const float *__restrict__ ln_c2)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x, h = blockIdx.y, dim = threadIdx.x;
    const int4 ri = row_info[r];
    if (ri.x < 0) return;
    const int d_model = n_heads * kHeadDim;
    const float2 st = ln_stats ? ln_stats[r] : make_float2(0.f, 1.f);
#pragma unroll
    for (int kv = 0; kv < 2; ++kv) {
        const int col = (1 + kv) * d_model + h * kHeadDim + dim;
        float y = qkv[(size_t)r * ldq + col];
        if (ln_stats) y = fmaf(st.y, y - st.x * ln_c1[col], ln_c2[col]);
        cache[((((size_t)ri.x * 2 + kv) * n_heads + h) * (size_t)seq_capacity + ri.y) * kHeadDim + dim] = from_f32<CT>(y);
    }
}

// End of a prefill chunk: every utterance has `chunk` more positions cached; after the last chunk the argmax of the
// last prompt position (rows 0 .. batch - 1) is handed out and becomes the utterance's current token.
__global__ void prefill_finish_kernel(DecState *state, const int32_t *__restrict__ active_list,
                                      unsigned long long *__restrict__ keys, int32_t *__restrict__ t_u, int chunk, int last,
                                      int32_t *__restrict__ next_out, int32_t *__restrict__ cur_tok)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= state->batch) return;
    const int u = active_list[r];
    t_u[u] += chunk;
    if (last) {
        const int32_t tok = argmax_key_index(keys[r]);
        keys[r] = 0ull;
        cur_tok[u] = tok;
        if (next_out) next_out[u] = tok;
    }
}

// ------------------------------------------------------------------------------------------------------------
// End of a step: decode the argmax keys, hand the choice out by utterance id, advance t_u, and (greedy mode)
// record the token, feed it back and retire finished utterances.
// ------------------------------------------------------------------------------------------------------------
__global__ void finish_step_kernel(DecState *state, const int32_t *__restrict__ active_list,
                                   unsigned long long *__restrict__ keys, int32_t *__restrict__ t_u,
                                   int32_t *__restrict__ next_out /* by utterance, nullable */,
                                   int greedy, int32_t *__restrict__ cur_tok, int32_t *__restrict__ retired,
                                   const int32_t *__restrict__ max_len, int eos_id,
                                   int32_t *__restrict__ tokens_out, int tokens_ld, int32_t *__restrict__ out_lens)
{
    AED_TRACE_BEGIN(state, 6);
    asm volatile("griddepcontrol.wait;" ::: "memory");       // launched with programmatic stream serialization
    int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= state->n_active) return;
    int u = active_list[r];
    int32_t tok = argmax_key_index(keys[r]);
    keys[r] = 0ull;
    int t = t_u[u];
    t_u[u] = t + 1;
    if (next_out) next_out[u] = tok;
    if (greedy) {
        cur_tok[u] = tok;
        tokens_out[(size_t)u * tokens_ld + t] = tok;
        if (t + 1 >= max_len[u] || (eos_id >= 0 && tok == eos_id)) {
            retired[u] = 1;
            out_lens[u] = t + 1;
            atomicAdd(&state->n_retired, 1);          // the host polls this to stop issuing steps once every utterance is done
        }
    }
}

// New utterances take over slots: position 0, start token, their encoder range and forced length.  One thread each.
constexpr int kMaxAdmit = 16;
struct AdmitBatch {
    int n;
    int slot[kMaxAdmit], n_frames[kMaxAdmit], frame0[kMaxAdmit], forced_len[kMaxAdmit];
};
__global__ void admit_slots_kernel(AdmitBatch b, int bos, int32_t *__restrict__ enc_len, int32_t *__restrict__ enc_off,
                                   int32_t *__restrict__ t_u, int32_t *__restrict__ retired, int32_t *__restrict__ cur_tok,
                                   int32_t *__restrict__ max_len, int32_t *__restrict__ out_lens)
{
    const int i = threadIdx.x;
    if (blockIdx.x != 0 || i >= b.n) return;
    const int slot = b.slot[i];
    enc_len[slot] = b.n_frames[i];
    enc_off[slot] = b.frame0[i];
    t_u[slot] = 0;
    cur_tok[slot] = bos;
    max_len[slot] = b.forced_len[i];
    if (out_lens) out_lens[slot] = 0;
    retired[slot] = 0;
}

__global__ void fill_i32_kernel(int32_t *p, int32_t v, size_t n)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

}  // namespace aed
