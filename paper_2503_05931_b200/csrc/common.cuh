// Shared device helpers for the AED decoder kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace aed {

constexpr int kHeadDim = 64;        // every supported model has head_dim 64
constexpr int kAttnChunk = 64;      // positions per flash-decoding work item
constexpr int kPartialStride = 66;  // floats per attention partial: max, sum, 64 accumulators

// Device-resident decode state (lives in the caller's workspace).
struct DecState {
    int32_t n_active;    // rows taking part in the current step
    int32_t error;       // sticky: 0 ok, 1 = a row would have overflowed the self-attention cache
    int32_t n_retired;   // utterances retired so far
    int32_t grid_sync;   // arrival counter of the persistent step kernel, cleared by the first kernel of a step
    int32_t batch;       // utterances of the current batch (written by the cross-K/V precompute)
};

// Optional device-side timeline (debug builds with -DAED_TRACE): block 0 of every traced kernel stamps its start
// time.  The buffer follows the decode state in the workspace.
struct TraceBuf {
    uint32_t count, pad;
    struct { uint32_t id, pad; unsigned long long t_ns; } ev[1 << 16];
};
#ifdef AED_TRACE
__device__ __forceinline__ void trace_begin(const DecState *state, uint32_t id)
{
    if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
        TraceBuf *tb = reinterpret_cast<TraceBuf *>(reinterpret_cast<char *>(const_cast<DecState *>(state)) + 256);
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        uint32_t i = atomicAdd(&tb->count, 1u);
        if (i < (1u << 16)) { tb->ev[i].id = id; tb->ev[i].t_ns = t; }
    }
}
// stamp from whichever thread of block 0 calls it
__device__ __forceinline__ void trace_mark(const DecState *state, uint32_t id)
{
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
        TraceBuf *tb = reinterpret_cast<TraceBuf *>(reinterpret_cast<char *>(const_cast<DecState *>(state)) + 256);
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        uint32_t i = atomicAdd(&tb->count, 1u);
        if (i < (1u << 16)) { tb->ev[i].id = id; tb->ev[i].t_ns = t; }
    }
}
// Cheap marks for one thread of block 0: a range of the buffer is reserved once (the atomic's latency is paid
// where nothing waits on it), later marks are plain stores.
struct TraceCursor { uint32_t next, end; };
__device__ __forceinline__ TraceCursor trace_reserve(const DecState *state, uint32_t n)
{
    TraceCursor c{0u, 0u};
    if (n > 0 && blockIdx.y == 0 && blockIdx.z == 0) {
        TraceBuf *tb = reinterpret_cast<TraceBuf *>(reinterpret_cast<char *>(const_cast<DecState *>(state)) + 256);
        c.next = atomicAdd(&tb->count, n);
        c.end = c.next + n;
        if (c.end > (1u << 16)) c.end = c.next;
    }
    return c;
}
// The SM's cycle counter (low 32 bits) goes with every mark; the global nanosecond timer, which costs a few hundred
// nanoseconds to read, only where asked for (the first mark of a kernel, to place it on the common axis).
template <bool kWallClock>
__device__ __forceinline__ void trace_put(const DecState *state, TraceCursor &c, uint32_t id)
{
    if (c.next < c.end) {
        TraceBuf *tb = reinterpret_cast<TraceBuf *>(reinterpret_cast<char *>(const_cast<DecState *>(state)) + 256);
        unsigned long long t = 0;
        if (kWallClock) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        tb->ev[c.next].id = id;
        tb->ev[c.next].pad = static_cast<uint32_t>(clock64());
        tb->ev[c.next].t_ns = t;
        ++c.next;
    }
}
#define AED_TRACE_BEGIN(state, id) trace_begin(state, id)
#define AED_TRACE_MARK(state, id) trace_mark(state, id)
#define AED_TRACE_RESERVE(cur, state, n) TraceCursor cur = trace_reserve(state, n)
#define AED_TRACE_PUT(state, cur, id) trace_put<false>(state, cur, id)
#define AED_TRACE_PUT_NS(state, cur, id) trace_put<true>(state, cur, id)
#else
#define AED_TRACE_BEGIN(state, id) ((void)0)
#define AED_TRACE_MARK(state, id) ((void)0)
#define AED_TRACE_RESERVE(cur, state, n) ((void)0)
#define AED_TRACE_PUT(state, cur, id) ((void)0)
#define AED_TRACE_PUT_NS(state, cur, id) ((void)0)
#endif

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 8 consecutive elements of type T, starting at a 16-byte (bf16) / 32-byte (fp32) aligned address, as floats.
__device__ __forceinline__ void load8(const float *p, float (&v)[8])
{
    float4 a = *reinterpret_cast<const float4 *>(p);
    float4 b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8])
{
    uint4 raw = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// 4 consecutive elements as floats (16-byte aligned for fp32, 8-byte aligned for bf16).
__device__ __forceinline__ void load4(const float *p, float (&v)[4])
{
    float4 a = *reinterpret_cast<const float4 *>(p);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16 *p, float (&v)[4])
{
    uint2 raw = *reinterpret_cast<const uint2 *>(p);
    v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xFFFF0000u);
    v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xFFFF0000u);
}

// One byte of the 8-bit floating-point format E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no
// infinities, largest finite value 448): the optional storage type of the cross-attention K/V store.
struct fp8e4m3 { uint8_t bits; };

// two floats -> two E4M3 bytes (lo in the low byte), round to nearest even, saturating at the largest finite value
__device__ __forceinline__ uint16_t pack_e4m3x2(float lo, float hi)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// two E4M3 bytes -> two floats (exact)
__device__ __forceinline__ float2 unpack_e4m3x2(uint16_t v)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(v));
    return __half22float2(*reinterpret_cast<__half2 *>(&h2));
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Monotone map float -> uint32 (larger float => larger key), used to take an argmax with integer atomics.
__device__ __forceinline__ uint32_t float_order_key(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// (value, index) packed so that the maximum key is the largest value and, among equals, the lowest index.
__device__ __forceinline__ unsigned long long argmax_key(float f, uint32_t idx)
{
    return (static_cast<unsigned long long>(float_order_key(f)) << 32) | (0xFFFFFFFFu - idx);
}
__device__ __forceinline__ int32_t argmax_key_index(unsigned long long key)
{
    return static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(key & 0xFFFFFFFFull));
}

}  // namespace aed
