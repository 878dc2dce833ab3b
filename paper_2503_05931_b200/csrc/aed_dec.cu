// Host side of the AED decoder library: handle, workspace layout, launch sequences, C ABI.
#include "../../include/aed_dec.h"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "step_kernels.cuh"
#include "tc_gemm.cuh"
#include "step_gemm.cuh"
#include "step_gemv.cuh"
#include "vocab_gemv.cuh"
#include "crosskv_gemm.cuh"
#include "stream_schedule.h"

using namespace aed;

namespace {

thread_local std::string g_create_error;

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Row counts are rounded up to 16, 32, ..., 256 and then to multiples of 256, so that few graphs cover a decode.
int rows_bucket(int rows)
{
    int b = 16;
    while (b < rows && b < 256) b <<= 1;
    if (b < rows) b = (rows + 255) / 256 * 256;
    return b;
}

// Row count a step graph is captured for.  Kernels whose grids follow the row count (attention: one block per row and
// head) pay for every row of the grid, also for those beyond the device-side count, whose blocks only find out that
// they have nothing to do; so the graphs are keyed finer than the power-of-two tiles of the projections: 4, then multiples
// of 8 up to 64 rows, of 16 up to 256, of 32 beyond.  Never above rows_bucket(rows).
int rows_key(int rows)
{
    if (rows <= 4) return 4;         // the projections of steps of at most 4 rows take a form of their own
    const int g = rows <= 64 ? 8 : rows <= 256 ? 16 : 32;
    return (rows + g - 1) / g * g;
}

struct LayerWeights {
    const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o;
    const void *ln2_g, *ln2_b, *w_q_c, *b_q_c, *w_kv_c, *b_kv_c, *w_o_c, *b_o_c;
    const void *ln3_g, *ln3_b, *w_ff1, *b_ff1, *w_ff2, *b_ff2;
};

// Byte offsets of every region of the caller's workspace.
struct Layout {
    size_t self_cache, cross_store, x, act, qkv, hid, partials, pe, keys, state;
    size_t t_u, retired, active_list, cur_tok, enc_off, enc_len, max_len, row_info, row_tok, len_order, total;
    size_t self_layer_elems, cross_layer_elems;
    int max_chunks;
    // bf16 mode: activation planes (high, low) that feed the tensor-core projections
    size_t actd_hi, actd_lo, actf_hi, actf_lo;
    size_t fold_c, ln_stats, qc;          // LayerNorm-fold constants per layer, row statistics (3 sets)
    size_t slot_tokens, slot_lens;        // aed_dec_decode_stream: token rows and lengths of the slots
    size_t fold_out;                      // c1 | c2 of the vocabulary projection with the final LayerNorm folded in
    size_t comp_w, comp_b;                // per layer: Wqc diag(gamma2) Wo as bf16 [d, d], and Wqc (gamma2 * bo) as fp32 [d]
    size_t ckv_maps, ckv_bias;            // per-layer tensor maps and bias pointers of the cross-K/V weights
    size_t fold_layer_floats;
    int rows_cap;
};

bool config_supported(const aed_dec_config_t &c, std::string *why)
{
    auto fail = [&](const char *m) { if (why) *why = m; return false; };
    if (c.n_layers < 1 || c.d_model < 1 || c.n_heads < 1 || c.d_ffn < 1 || c.vocab < 2 || c.d_enc < 1)
        return fail("model dimensions must be positive (vocab >= 2)");
    if (c.dtype != AED_DTYPE_F32 && c.dtype != AED_DTYPE_BF16) return fail("dtype must be AED_DTYPE_F32 or AED_DTYPE_BF16");
    if (c.max_batch < 1 || c.max_total_enc_frames < 1 || c.max_enc_len < 1 || c.max_dec_len < 1)
        return fail("capacities must be positive");
    if (c.max_enc_len > c.max_total_enc_frames) return fail("max_enc_len exceeds max_total_enc_frames");
    if (!(c.ln_eps > 0.f)) return fail("ln_eps must be positive");
    if (c.cross_kv_format != AED_CROSS_KV_DTYPE && c.cross_kv_format != AED_CROSS_KV_E4M3)
        return fail("cross_kv_format must be AED_CROSS_KV_DTYPE or AED_CROSS_KV_E4M3");
    return true;
}

bool shape_supported(const aed_dec_config_t &c, std::string *why)
{
    auto fail = [&](const char *m) { if (why) *why = m; return false; };
    if (c.d_model % c.n_heads != 0 || c.d_model / c.n_heads != kHeadDim) return fail("head_dim must be 64");
    if (c.d_model % 64 || c.d_ffn % 64 || c.d_enc % 64) return fail("d_model, d_ffn and d_enc must be multiples of 64");
    if (c.d_model > 8192) return fail("d_model above 8192 is not supported");
    if (c.cross_kv_format == AED_CROSS_KV_E4M3 && c.dtype != AED_DTYPE_BF16)
        return fail("the 8-bit cross-attention K/V store needs the bf16 configuration");
    return true;
}

Layout make_layout(const aed_dec_config_t &c)
{
    Layout L{};
    const size_t e = c.dtype == AED_DTYPE_BF16 ? 2 : 4;
    const size_t B = c.max_batch, d = c.d_model, F = c.d_ffn;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    L.self_layer_elems = B * 2 * d * (size_t)c.max_dec_len;
    L.cross_layer_elems = 2 * d * (size_t)c.max_total_enc_frames;
    L.self_cache = take(L.self_layer_elems * c.n_layers * e);
    L.cross_store = take(L.cross_layer_elems * c.n_layers * (c.cross_kv_format == AED_CROSS_KV_E4M3 ? 1 : e));
    L.x = take(B * d * 4);
    L.act = take(B * (d > F ? d : F) * 4);
    L.qkv = take(B * 3 * d * 4);
    L.hid = take(B * F * 4);
    int longest = c.max_enc_len > c.max_dec_len ? c.max_enc_len : c.max_dec_len;
    L.max_chunks = (longest + kAttnChunk - 1) / kAttnChunk;
    L.partials = take(B * c.n_heads * (size_t)L.max_chunks * kPartialStride * 4);
    L.pe = take((size_t)c.max_dec_len * d * 4);
    L.keys = take(B * 8);
    L.state = take(sizeof(DecState));
#ifdef AED_TRACE
    take(sizeof(TraceBuf));       // must directly follow the state (see trace_begin)
#endif
    L.t_u = take(B * 4);
    L.retired = take(B * 4);
    L.active_list = take(B * 4);
    L.cur_tok = take(B * 4);
    L.enc_off = take((B + 1) * 4);
    L.enc_len = take(B * 4);
    L.max_len = take(B * 4);
    L.row_info = take((size_t)rows_bucket(c.max_batch) * 16);      // grids are sized for the bucket
    L.row_tok = take((size_t)rows_bucket(c.max_batch) * 4);        // prefill: the token of every (utterance, position) row
    L.len_order = take(B * 4);                                     // utterances by decreasing encoder length
    L.rows_cap = (int)align_up(B, 16);
    L.slot_tokens = take(B * (size_t)c.max_dec_len * 4);
    L.slot_lens = take(B * 4);
    if (c.dtype == AED_DTYPE_BF16) {
        L.actd_hi = take((size_t)L.rows_cap * d * 2);
        L.actd_lo = take((size_t)L.rows_cap * d * 2);
        L.actf_hi = take((size_t)L.rows_cap * F * 2);        // FFN hidden layer as planes (steps with many rows)
        L.actf_lo = take((size_t)L.rows_cap * F * 2);
        L.fold_layer_floats = 2 * (3 * d + d + F);       // c1 | c2 for qkv, then for cross-q, then for ffn1
        L.fold_c = take(L.fold_layer_floats * c.n_layers * 4);
        L.ln_stats = take((size_t)3 * rows_bucket(c.max_batch) * 8);
        L.qc = take(B * d * 4);
        L.ckv_maps = take((size_t)c.n_layers * sizeof(CUtensorMap));
        L.ckv_bias = take((size_t)c.n_layers * sizeof(void *));
        L.fold_out = take((size_t)2 * c.vocab * 4);
        L.comp_w = take((size_t)c.n_layers * d * d * 2);
        L.comp_b = take((size_t)c.n_layers * d * 4);
    }
    L.total = off;
    return L;
}

}  // namespace

struct aed_dec {
    aed_dec_config_t cfg;
    Layout lay;
    cudaStream_t stream;
    char *ws;
    // borrowed weights
    const void *embed, *final_ln_g, *final_ln_b, *w_out, *b_out;
    std::vector<LayerWeights> layers;
    // host view of the current batch
    int batch = 0;
    bool have_batch = false;
    bool fresh_batch = false;       // no step issued since the precompute
    int steps_issued = 0;           // steps of any kind since the precompute: upper bound on any t_u
    int full_steps = 0;             // steps without a mask: lower bound on t_u of every utterance not retired
    int total_frames = 0;
    std::vector<int32_t> enc_len, enc_off;
    // continuous batching: the batch is a set of slots that utterances enter and leave one by one
    bool slot_mode = false;
    std::vector<int32_t> slot_t, slot_max;      // steps issued since the slot's utterance entered (-1: empty), its forced length
    std::string err;
    int64_t launches = 0;
    // optional per-kernel-family timing (CUDA events around every launch)
    bool profiling = false;
    std::vector<cudaEvent_t> prof_events;          // pool, two per recorded launch
    std::vector<int> prof_family;                  // family of each recorded launch
    size_t prof_used = 0;
    // bf16 mode: TMA descriptors of the weight matrices and of the activation planes (one per MMA N in 16..256)
    struct TcLayerMaps { CUtensorMap qkv, o, qc, oc, ff1, ff2, o_qc; };      // o_qc: the composite Wqc diag(gamma2) Wo
    std::vector<TcLayerMaps> tc_layers;
    CUtensorMap tc_w_out;
    CUtensorMap tc_actd[5][2], tc_actf[5][2];     // [log2(N/16)][plane]: activation planes [rows, d] and [rows, F]
    CUtensorMap tc_src_x[5], tc_src_att[5], tc_src_hid[5];   // fp32 sources of the fused projections, per MMA N
    bool use_tc = false;
    int sm_count = 148;
    int tc_target_ctas = 128;
    bool tc_target_fixed = false;         // set from the environment: use tc_target_ctas at every row count
    bool use_pdl = true;
    bool attn_pipe = true;
    bool use_gemv = true;           // steps of few rows: projections by warp-level MMAs (step_gemv.cuh)
    int gemv_rows = 64;             // ... up to this many rows
    int gemv_direct_rows = 4;       // ... with the activation fragments straight from global memory up to this many
    int planes_rows = 128;                // steps with more rows make their activation planes once per projection input
    // greedy decoding replays one captured CUDA graph per (row bucket, self-attention chunk count, output buffers)
    typedef std::tuple<int, int, const void *, const void *> GraphKey;
    struct GraphEntry { cudaGraphExec_t exec; int64_t nodes; };
    std::map<GraphKey, GraphEntry> graphs;
    cudaStream_t capture_stream = nullptr;
    bool use_graphs = true;
    // set only while aed_dec_step_static_scratch runs: attention partials go here instead of the workspace
    float *partials_override = nullptr;
    // greedy decoding with an end-of-sequence id: the retired count of recent steps, copied to pinned host memory
    static constexpr int kProbeSlots = 16;
    int32_t *probe_host = nullptr;
    cudaEvent_t probe_event[kProbeSlots] = {};

    template <typename T> T *at(size_t off) const { return reinterpret_cast<T *>(ws + off); }
    DecState *state() const { return at<DecState>(lay.state); }
};

namespace {

aed_status_t fail(aed_dec *d, aed_status_t code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (d) d->err = buf; else g_create_error = buf;
    return code;
}

#define AED_CUDA(dec, expr)                                                                              \
    do {                                                                                                 \
        cudaError_t e__ = (expr);                                                                        \
        if (e__ != cudaSuccess) return fail(dec, AED_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

#define AED_LAUNCHED(dec)                                                                                      \
    do {                                                                                                       \
        (dec)->launches++;                                                                                     \
        cudaError_t e__ = cudaGetLastError();                                                                  \
        if (e__ != cudaSuccess) return fail(dec, AED_ERR_CUDA, "kernel launch failed at %s:%d: %s", __FILE__, \
                                            __LINE__, cudaGetErrorString(e__));                               \
    } while (0)

enum KernelFamily { KF_BOOKKEEPING = 0, KF_EMBED, KF_LAYERNORM, KF_GEMM_QKV, KF_ATTN_SELF, KF_ATTN_COMBINE, KF_GEMM_O,
                    KF_GEMM_QC, KF_ATTN_CROSS, KF_GEMM_OC, KF_GEMM_FF1, KF_GEMM_FF2, KF_GEMM_VOCAB, KF_PRECOMPUTE,
                    KF_COUNT };
const char *const kFamilyNames[KF_COUNT] = {"bookkeeping", "embed", "layernorm", "gemm_qkv", "attn_self", "attn_combine",
                                            "gemm_o", "gemm_qc", "attn_cross", "gemm_oc", "gemm_ff1", "gemm_ff2",
                                            "gemm_vocab", "precompute_cross_kv"};
// The projections of steps with few rows run in kernels of their own (step_gemv.cuh); the profile keeps the call site
// and says which kernel ran it: family + KF_COUNT * variant, reported as "gemm_qkv@gemv", "gemm_qkv@gemv_staged".
enum { KV_TCGEN05 = 0, KV_GEMV = 1, KV_GEMV_STAGED = 2, KV_COUNT = 3 };
const char *const kVariantSuffix[KV_COUNT] = {"", "@gemv", "@gemv_staged"};

// Records an event before and after the launches issued while it is alive (profiling mode only).
struct ProfScope {
    aed_dec *dec;
    bool on;
    ProfScope(aed_dec *d, int family) : dec(d), on(d->profiling)
    {
        if (!on) return;
        if (dec->prof_used + 2 > dec->prof_events.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
                dec->prof_events.push_back(e);
            }
        }
        dec->prof_family.push_back(family);
        cudaEventRecord(dec->prof_events[dec->prof_used], dec->stream);
    }
    ~ProfScope()
    {
        if (!on) return;
        cudaEventRecord(dec->prof_events[dec->prof_used + 1], dec->stream);
        dec->prof_used += 2;
    }
};

// ---- typed launch sequences ------------------------------------------------------------------------------

template <typename T>
aed_status_t launch_layernorm(aed_dec *dec, int rows_ub, const float *x, const void *g, const void *b, float *out)
{
    ProfScope ps(dec, KF_LAYERNORM);
    const int d = dec->cfg.d_model;
    if (d <= 2048)
        layernorm_kernel<T, 8><<<rows_ub, 256, 0, dec->stream>>>(dec->state(), x, (const T *)g, (const T *)b, d,
                                                                 dec->cfg.ln_eps, out);
    else
        layernorm_kernel<T, 8><<<rows_ub, 1024, 0, dec->stream>>>(dec->state(), x, (const T *)g, (const T *)b, d,
                                                                  dec->cfg.ln_eps, out);
    AED_LAUNCHED(dec);
    return AED_OK;
}

template <typename AT, typename T, int EPI>
aed_status_t launch_gemm(aed_dec *dec, int family, int rows_ub, int rows_fixed, const AT *A, int lda, const void *W,
                         const void *bias, int M, int K, const GemmEpilogueArgs<T> &ep)
{
    ProfScope ps(dec, family);
    dim3 grid((M + 31) / 32, (rows_ub + 63) / 64);
    gemm_rows_kernel<AT, T, T, EPI><<<grid, 128, 0, dec->stream>>>(dec->state(), rows_fixed, A, lda, (const T *)W,
                                                                    (const T *)bias, M, K, ep);
    AED_LAUNCHED(dec);
    return AED_OK;
}

template <typename T, bool kCross, bool kAppend = false>
aed_status_t launch_attention(aed_dec *dec, int rows_ub, int len_ub, const float *q, int ldq, const T *cache,
                              int seq_capacity, float *out)
{
    const auto &c = dec->cfg;
    const int H = c.n_heads;
    int chunks_ub = (len_ub + kAttnChunk - 1) / kAttnChunk;
    if (chunks_ub > dec->lay.max_chunks) chunks_ub = dec->lay.max_chunks;
    dim3 grid(rows_ub * H, (chunks_ub + 3) / 4);
    float *partials = dec->partials_override ? dec->partials_override : dec->at<float>(dec->lay.partials);
    {
    ProfScope ps(dec, kCross ? KF_ATTN_CROSS : KF_ATTN_SELF);
    attn_partial_kernel<T, kCross, kAppend><<<grid, 128, 0, dec->stream>>>(
        dec->state(), dec->at<int32_t>(dec->lay.active_list), q, ldq, const_cast<T *>(cache), H, seq_capacity,
        dec->at<int32_t>(dec->lay.t_u), dec->at<int32_t>(dec->lay.enc_off), dec->at<int32_t>(dec->lay.enc_len),
        dec->lay.max_chunks, 1.0f / sqrtf((float)kHeadDim), partials);
    AED_LAUNCHED(dec);
    }
    ProfScope ps(dec, KF_ATTN_COMBINE);
    attn_combine_kernel<kCross><<<(rows_ub * H + 3) / 4, 128, 0, dec->stream>>>(
            dec->state(), dec->at<int32_t>(dec->lay.active_list), partials, H, dec->at<int32_t>(dec->lay.t_u),
        dec->at<int32_t>(dec->lay.enc_len), dec->lay.max_chunks, out, c.d_model);
    AED_LAUNCHED(dec);
    return AED_OK;
}

// Attention in one kernel per call (no scratch): one block per (row, head), one warp per 16 positions, at most 8.
// The kernel starts with a programmatic-dependency wait, so it may be launched ahead of its predecessor's end.
template <typename T, bool kCross, bool kAppend>
aed_status_t launch_attention_fused(aed_dec *dec, int rows_ub, int len_ub, const float *q, int ldq, const T *cache,
                                    int seq_capacity, float *out, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                    const float2 *ln_stats = nullptr, const float *ln_c1 = nullptr,
                                    const float *ln_c2 = nullptr, bool pdl = false, const float *stats_x = nullptr)
{
    ProfScope ps(dec, kCross ? KF_ATTN_CROSS : KF_ATTN_SELF);
    int warps = (len_ub + fused_chunk<T>() - 1) / fused_chunk<T>();
    if (warps < 2) warps = 2;                    // at least 64 threads: the merge uses one thread per head dimension
    if (warps > kFusedMaxWarps) warps = kFusedMaxWarps;
    // Attention starts early (programmatic launch) and holds each warp's first chunk in registers; rows longer than
    // 8 x 16 positions loop and find their later chunks prefetched in L2.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(rows_ub * dec->cfg.n_heads);
    cfg.blockDim = dim3(warps * 32);
    cfg.stream = dec->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // Few blocks with long rows (late steps): the software-pipelined variant, two blocks per SM hold the whole grid.
    const bool pipe = kCross && !kAppend && rows_ub * dec->cfg.n_heads <= 2 * dec->sm_count && dec->attn_pipe;
    auto kernel = pipe ? attn_fused_kernel<T, kCross, kAppend, kCross && !kAppend> : attn_fused_kernel<T, kCross, kAppend, false>;
    if constexpr (kCross && !kAppend) {
        if (stats_x) kernel = pipe ? attn_fused_kernel<T, true, false, true, true> : attn_fused_kernel<T, true, false, false, true>;
    }
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, (const DecState *)dec->state(),
                                       (const int4 *)dec->at<int4>(dec->lay.row_info), q, ldq, const_cast<T *>(cache),
                                       dec->cfg.n_heads, seq_capacity, 1.0f / sqrtf((float)kHeadDim), out, out_hi, out_lo,
                                       dec->cfg.d_model, ln_stats, ln_c1, ln_c2, stats_x, dec->cfg.ln_eps);
    if (e != cudaSuccess) return fail(dec, AED_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    AED_LAUNCHED(dec);
    return AED_OK;
}

// A launch that may start before its predecessor in the stream has ended (programmatic stream serialization): the
// kernel itself waits (griddepcontrol.wait) before it touches what the predecessor wrote.
aed_status_t launch_pdl_impl(aed_dec *dec, const void *kernel, dim3 grid, dim3 block, size_t smem, void **args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = dec->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = dec->use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelExC(&cfg, kernel, args);
    if (e != cudaSuccess) return fail(dec, AED_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
    AED_LAUNCHED(dec);
    return AED_OK;
}

#define AED_TRY(expr)                        \
    do {                                     \
        aed_status_t s__ = (expr);           \
        if (s__ != AED_OK) return s__;       \
    } while (0)

// The forward pass of one step for the rows in the active list (at most rows_ub of them).
//   tokens: by utterance.  self_len_ub: upper bound on t_u + 1.
template <typename T>
aed_status_t forward_step(aed_dec *dec, int rows_ub, int self_len_ub, const int32_t *tokens, float *logits_out)
{
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    const int d = c.d_model, F = c.d_ffn, V = c.vocab;
    float *x = dec->at<float>(L.x), *act = dec->at<float>(L.act), *qkv = dec->at<float>(L.qkv), *hid = dec->at<float>(L.hid);
    const int32_t *active_list = dec->at<int32_t>(L.active_list), *t_u = dec->at<int32_t>(L.t_u);

    {
        ProfScope ps(dec, KF_EMBED);
        embed_kernel<T><<<rows_ub, 256, 0, dec->stream>>>(dec->state(), active_list, tokens, t_u, (const T *)dec->embed,
                                                          dec->at<float>(L.pe), d, V, sqrtf((float)d), x);
        AED_LAUNCHED(dec);
    }

    GemmEpilogueArgs<T> ep{};
    ep.active_list = active_list;
    ep.t_u = t_u;
    ep.max_dec_len = c.max_dec_len;
    ep.d_model = d;
    ep.n_heads = c.n_heads;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = dec->layers[l];
        T *self_cache = dec->at<T>(L.self_cache) + (size_t)l * L.self_layer_elems;
        const T *cross = dec->at<T>(L.cross_store) + (size_t)l * L.cross_layer_elems;
        // masked self-attention
        AED_TRY(launch_layernorm<T>(dec, rows_ub, x, w.ln1_g, w.ln1_b, act));
        ep.out = qkv; ep.ldo = d; ep.self_cache = self_cache;
        AED_TRY((launch_gemm<float, T, EPI_QKV>(dec, KF_GEMM_QKV, rows_ub, -1, act, d, w.w_qkv, w.b_qkv, 3 * d, d, ep)));
        AED_TRY((launch_attention<T, false>(dec, rows_ub, self_len_ub, qkv, d, self_cache, c.max_dec_len, act)));
        ep.out = x; ep.ldo = d;
        AED_TRY((launch_gemm<float, T, EPI_RESID>(dec, KF_GEMM_O, rows_ub, -1, act, d, w.w_o, w.b_o, d, d, ep)));
        // cross-attention over the utterance's own encoder frames
        AED_TRY(launch_layernorm<T>(dec, rows_ub, x, w.ln2_g, w.ln2_b, act));
        ep.out = qkv; ep.ldo = d;
        AED_TRY((launch_gemm<float, T, EPI_STORE>(dec, KF_GEMM_QC, rows_ub, -1, act, d, w.w_q_c, w.b_q_c, d, d, ep)));
        AED_TRY((launch_attention<T, true>(dec, rows_ub, c.max_enc_len, qkv, d, cross, c.max_total_enc_frames, act)));
        ep.out = x; ep.ldo = d;
        AED_TRY((launch_gemm<float, T, EPI_RESID>(dec, KF_GEMM_OC, rows_ub, -1, act, d, w.w_o_c, w.b_o_c, d, d, ep)));
        // feed-forward
        AED_TRY(launch_layernorm<T>(dec, rows_ub, x, w.ln3_g, w.ln3_b, act));
        ep.out = hid; ep.ldo = F;
        AED_TRY((launch_gemm<float, T, EPI_RELU>(dec, KF_GEMM_FF1, rows_ub, -1, act, d, w.w_ff1, w.b_ff1, F, d, ep)));
        ep.out = x; ep.ldo = d;
        AED_TRY((launch_gemm<float, T, EPI_RESID>(dec, KF_GEMM_FF2, rows_ub, -1, hid, F, w.w_ff2, w.b_ff2, d, F, ep)));
    }
    AED_TRY(launch_layernorm<T>(dec, rows_ub, x, dec->final_ln_g, dec->final_ln_b, act));
    ep.logits_out = logits_out;
    ep.keys = dec->at<unsigned long long>(L.keys);
    AED_TRY((launch_gemm<float, T, EPI_LOGITS>(dec, KF_GEMM_VOCAB, rows_ub, -1, act, d, dec->w_out, dec->b_out, V, d, ep)));
    return AED_OK;
}


// ---- tensor-core path (bf16 mode) ----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// matrix [rows, cols] row-major; box = box_rows x 64 columns, zero fill out of bounds.  bf16 operands use the
// 128-byte swizzle the MMA descriptors name; fp32 staging tiles are copied unswizzled.
bool encode_map(CUtensorMap *map, const void *base, size_t rows, size_t cols, int box_rows, bool fp32 = false)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const size_t esz = fp32 ? 4 : 2;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * esz};
    cuuint32_t box[2] = {(cuuint32_t)tc::kBlockK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              fp32 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kTcSmemBudget = 200 * 1024;

aed_status_t tc_setup(aed_dec *dec)
{
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    const size_t d = c.d_model, F = c.d_ffn;
    if (!encode_tiled_fn()) return fail(nullptr, AED_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    bool ok = true;
    dec->tc_layers.resize(c.n_layers);
    std::vector<CUtensorMap> kvc_maps(c.n_layers);
    std::vector<const void *> kvc_bias(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = dec->layers[l];
        aed_dec::TcLayerMaps &m = dec->tc_layers[l];
        ok = ok && encode_map(&m.qkv, w.w_qkv, 3 * d, d, tc::kTileM) && encode_map(&m.o, w.w_o, d, d, tc::kTileM) &&
             encode_map(&m.qc, w.w_q_c, d, d, tc::kTileM) && encode_map(&m.oc, w.w_o_c, d, d, tc::kTileM) &&
             encode_map(&m.ff1, w.w_ff1, F, d, tc::kTileM) && encode_map(&m.ff2, w.w_ff2, d, F, tc::kTileM) &&
             encode_map(&kvc_maps[l], w.w_kv_c, 2 * d, c.d_enc, ckv::kTileN) &&
             encode_map(&m.o_qc, dec->ws + L.comp_w + (size_t)l * d * d * 2, d, d, tc::kTileM);
        kvc_bias[l] = w.b_kv_c;
    }
    ok = ok && encode_map(&dec->tc_w_out, dec->w_out, c.vocab, d, tc::kTileM);
    for (int i = 0; i < 5; ++i) {
        const int box = 16 << i;
        ok = ok && encode_map(&dec->tc_actd[i][0], dec->ws + L.actd_hi, L.rows_cap, d, box) &&
             encode_map(&dec->tc_actd[i][1], dec->ws + L.actd_lo, L.rows_cap, d, box) &&
             encode_map(&dec->tc_actf[i][0], dec->ws + L.actf_hi, L.rows_cap, F, box) &&
             encode_map(&dec->tc_actf[i][1], dec->ws + L.actf_lo, L.rows_cap, F, box) &&
             encode_map(&dec->tc_src_x[i], dec->ws + L.x, c.max_batch, d, box, true) &&
             encode_map(&dec->tc_src_att[i], dec->ws + L.act, c.max_batch, d, box, true) &&
             encode_map(&dec->tc_src_hid[i], dec->ws + L.hid, c.max_batch, F, box, true);
    }
    if (!ok) return fail(nullptr, AED_ERR_CUDA, "cuTensorMapEncodeTiled failed (are all weight tensors 16-byte aligned?)");
    const int smem = kTcSmemBudget + 1024;
    cudaError_t e = cudaFuncSetAttribute(tc::tc_gemm_kernel<tc::TC_EPI_LOGITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv::crosskv_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ckv::kStages * ckv::kStageBytes + 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv::crosskv_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ckv::kStages * ckv::kStageBytes + 1024);
    // tensor maps and bias pointers of the cross-K/V weights: read by the precompute kernel from the workspace
    if (e == cudaSuccess) e = cudaMemcpyAsync(dec->ws + L.ckv_maps, kvc_maps.data(), kvc_maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, dec->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dec->ws + L.ckv_bias, kvc_bias.data(), kvc_bias.size() * sizeof(void *), cudaMemcpyHostToDevice, dec->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(dec->stream);       // the host vectors go away
    int dev = 0, sms = 0;
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return fail(nullptr, AED_ERR_CUDA, "tensor-core path set-up: %s", cudaGetErrorString(e));
    dec->sm_count = sms > 0 ? sms : 148;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sg::step_gemm_kernel<sg::B_PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sg::step_gemm_kernel<sg::B_GAMMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sg::step_gemm_kernel<sg::B_LN_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sg::step_gemm_kernel<sg::B_PLANES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_PLAIN, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_GAMMA, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_LN_RELU, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_PLAIN, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4, 4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_GAMMA, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4, 4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sv::step_gemv_staged_kernel<sg::B_LN_RELU, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sv::sv_staged_smem(4, 4));

    if (e != cudaSuccess) return fail(nullptr, AED_ERR_CUDA, "tensor-core path set-up: %s", cudaGetErrorString(e));
    // LayerNorm-fold constants of every layer
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = dec->layers[l];
        float *fc = dec->at<float>(L.fold_c) + (size_t)l * L.fold_layer_floats;
        typedef __nv_bfloat16 T;
        sg::ln_fold_constants_kernel<<<(3 * d + 7) / 8, 256, 0, dec->stream>>>((const T *)w.w_qkv, (const T *)w.ln1_g, (const T *)w.ln1_b,
                                                                               (const T *)w.b_qkv, 3 * (int)d, (int)d, fc, fc + 3 * d);
        sg::ln_fold_constants_kernel<<<(d + 7) / 8, 256, 0, dec->stream>>>((const T *)w.w_q_c, (const T *)w.ln2_g, (const T *)w.ln2_b,
                                                                           (const T *)w.b_q_c, (int)d, (int)d, fc + 6 * d, fc + 7 * d);
        sg::ln_fold_constants_kernel<<<(F + 7) / 8, 256, 0, dec->stream>>>((const T *)w.w_ff1, (const T *)w.ln3_g, (const T *)w.ln3_b,
                                                                           (const T *)w.b_ff1, (int)F, (int)d, fc + 8 * d, fc + 8 * d + F);
        // The self-attention output projection and the cross-attention query projection meet without a nonlinearity:
        // their composite lets one launch run both (see forward_step_fused).
        T *cw = dec->at<T>(L.comp_w) + (size_t)l * d * d;
        float *cb = dec->at<float>(L.comp_b) + (size_t)l * d;
        sg::compose_weights_kernel<<<dim3((unsigned)((d + 15) / 16), (unsigned)((d + 15) / 16)), 256, 0, dec->stream>>>(
            (const T *)w.w_q_c, (const T *)w.ln2_g, (const T *)w.w_o, (int)d, cw);
        sg::compose_bias_kernel<<<(d + 7) / 8, 256, 0, dec->stream>>>((const T *)w.w_q_c, (const T *)w.ln2_g, (const T *)w.b_o, (int)d, cb);
        dec->launches += 5;
    }
    {
        typedef __nv_bfloat16 T;
        float *fo = dec->at<float>(L.fold_out);
        sg::ln_fold_constants_kernel<<<(c.vocab + 7) / 8, 256, 0, dec->stream>>>((const T *)dec->w_out, (const T *)dec->final_ln_g, (const T *)dec->final_ln_b,
                                                                                (const T *)dec->b_out, c.vocab, (int)d, fo, fo + c.vocab);
        dec->launches += 1;
    }
    e = cudaGetLastError();
    if (e == cudaSuccess && vg::vg_smem((int)d) <= 227 * 1024)
        e = cudaFuncSetAttribute(vg::vocab_gemv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, vg::vg_smem((int)d));
    if (e != cudaSuccess) return fail(nullptr, AED_ERR_CUDA, "fold constants: %s", cudaGetErrorString(e));
    {
        const char *v = getenv("AED_DEC_NO_PDL");
        dec->use_pdl = !(v && v[0] == '1');
        v = getenv("AED_DEC_NO_ATTN_PIPE");
        dec->attn_pipe = !(v && v[0] == '1');
        v = getenv("AED_DEC_NO_GEMV");
        dec->use_gemv = !(v && v[0] == '1');
        v = getenv("AED_DEC_GEMV_ROWS");
        if (v && atoi(v) >= 1 && atoi(v) <= 64) dec->gemv_rows = atoi(v);
        v = getenv("AED_DEC_GEMV_DIRECT_ROWS");
        if (v && atoi(v) >= 0 && atoi(v) <= 8) dec->gemv_direct_rows = atoi(v);
        v = getenv("AED_DEC_PLANES_ROWS");
        if (v && atoi(v) > 0) dec->planes_rows = atoi(v);

    }
    const char *ctas = getenv("AED_DEC_GEMM_CTAS");
    if (ctas && atoi(ctas) > 0) { dec->tc_target_ctas = atoi(ctas); dec->tc_target_fixed = true; }
    dec->use_tc = true;
    return AED_OK;
}

// MMA N for a step with at most rows_ub rows: the smallest of 16, 32, ..., 256 that covers them (or 256).
int tc_n_index(int rows_ub)
{
    int i = 0;
    while (i < 4 && (16 << i) < rows_ub) ++i;
    return i;
}

// The vocabulary projection on tensor cores: logits[r, v] = sum_k act[r, k] * Wout[v, k] (+ bias), argmax in the epilogue.
aed_status_t launch_vocab_gemm(aed_dec *dec, int rows_ub, tc::TcParams p, int rows_fixed = -1)
{
    ProfScope ps(dec, KF_GEMM_VOCAB);
    const int M = dec->cfg.vocab, K = dec->cfg.d_model;
    const int ni = tc_n_index(rows_ub), n_tile = 16 << ni;
    const int row_tiles = (rows_ub + n_tile - 1) / n_tile, m_tiles = (M + tc::kTileM - 1) / tc::kTileM;
    const int k_blocks = K / tc::kBlockK;
    p.a_rows = M;
    p.n_tile = n_tile;
    p.k_blocks = k_blocks;
    p.use_lo = 1;
    p.rows_fixed = rows_fixed;          // >= 0: only that many rows (a prefill pass projects its last-position rows only)
    p.state = dec->state();
    const int stage_bytes = tc::kATileBytes + 2 * n_tile * tc::kBlockK * 2;
    int stages = kTcSmemBudget / stage_bytes;
    if (stages > tc::kMaxStages) stages = tc::kMaxStages;
    if (stages > k_blocks) stages = k_blocks;
    // every ring stage belongs to one issuing thread: as many producers as stages (at most one per producer warp)
    int producers = stages >= tc::kProducerWarps ? tc::kProducerWarps : stages;
    stages -= stages % producers;
    const CUtensorMap *acts = dec->tc_actd[ni];
    dim3 grid(m_tiles, 1, row_tiles);
    void *args[] = {(void *)&dec->tc_w_out, (void *)&acts[0], (void *)&acts[1], &p, &stages, (void *)&producers};
    return launch_pdl_impl(dec, (const void *)tc::tc_gemm_kernel<tc::TC_EPI_LOGITS>, grid, dim3(tc::kThreads),
                           (size_t)stages * stage_bytes + 1024, args);
}

aed_status_t launch_pdl_impl(aed_dec *dec, const void *kernel, dim3 grid, dim3 block, size_t smem, void **args);

aed_status_t launch_ln_planes(aed_dec *dec, int rows_ub, const float *x, const void *g, const void *b, float *zero_buf,
                              int zero_cols)
{
    ProfScope ps(dec, KF_LAYERNORM);
    int d = dec->cfg.d_model;
    float eps = dec->cfg.ln_eps;
    const Layout &L = dec->lay;
    const DecState *state = dec->state();
    const __nv_bfloat16 *gp = (const __nv_bfloat16 *)g, *bp = (const __nv_bfloat16 *)b;
    __nv_bfloat16 *hi = dec->at<__nv_bfloat16>(L.actd_hi), *lo = dec->at<__nv_bfloat16>(L.actd_lo);
    void *args[] = {&state, &x, &gp, &bp, &d, &eps, &hi, &lo, &zero_buf, &zero_cols};
    return launch_pdl_impl(dec, (const void *)layernorm_planes_kernel<8>, dim3(rows_ub), dim3(d <= 2048 ? 256 : 1024), 0, args);
}

// ---- fused step (bf16 mode): 7 kernels per layer, chained with programmatic dependent launch -------------------

struct FusedGemm {
    const CUtensorMap *map;
    int M, K, mode;
};

template <int MODE>
aed_status_t launch_step_gemm(aed_dec *dec, int family, const CUtensorMap &map_w, const CUtensorMap *src_maps, int M,
                              int K, int rows_ub, sg::StepGemmParams p, const CUtensorMap (*plane_maps)[2] = nullptr,
                              const CUtensorMap *map_w2 = nullptr, int M2 = 0)
{
    // map_w2, M2: a second weight matrix [M2, K] over the same rows (its output, gamma and bias are in p)
    // plane_maps (B_PLANES only): [log2(N/16)][high, low] tensor maps of the ready-made activation planes
    // Rows per CTA tile: up to 128 (two ring stages still fit beside the transposition buffer); more rows are
    // covered by row tiles that re-read the weight tile from L2.
    int ni = tc_n_index(rows_ub);
    if (ni > 3) ni = 3;
    const int n_tile = 16 << ni;
    const int m_tiles1 = (M + tc::kTileM - 1) / tc::kTileM;
    const int row_tiles = (rows_ub + n_tile - 1) / n_tile, m_tiles = m_tiles1 + (map_w2 ? (M2 + tc::kTileM - 1) / tc::kTileM : 0);
    p.tiles_first = map_w2 ? m_tiles1 : 0;
    p.a_rows2 = M2;
    const int k_blocks = K / tc::kBlockK;
    const int stage_bytes = tc::kATileBytes + 2 * n_tile * tc::kBlockK * 2 + (MODE == sg::B_PLANES ? 0 : n_tile * tc::kBlockK * 4);
    int stages = kTcSmemBudget / stage_bytes;
    if (stages > sg::kMaxKb) stages = sg::kMaxKb;
    // k-splits: every split adds rows x features x 4 bytes of red.global traffic, so large batches stop at about
    // one CTA per SM.  Up to 64 rows that traffic is small, and CTAs with one or two k-blocks need so little
    // shared memory that the CTAs of the next projection become resident beside them and fetch their weight
    // tiles while this one still runs: there twice as many CTAs are worth it (measured on the 24-layer batch-64
    // workload: 129 ms per pass with a target of 128 CTAs, 121 ms with 256, 147 ms with 384).
    const int target_ctas = dec->tc_target_fixed ? dec->tc_target_ctas : (rows_ub <= 64 ? 256 : 128);
    int splits = target_ctas / (m_tiles * row_tiles);
    if (splits < 1) splits = 1;
    if (splits > k_blocks) splits = k_blocks;
    const int kb_max = (k_blocks + splits - 1) / splits;
    if (stages > kb_max) stages = kb_max;
    p.stages = stages;
    p.src_rows = dec->cfg.max_batch;
    p.a_rows = M;
    p.k_blocks = k_blocks;
    p.n_tile = n_tile;
    p.state = dec->state();
    p.eps = dec->cfg.ln_eps;
    // (41 to 64 rows: two row halves on grid.z and half the k-splits, up to four k-blocks per CTA.  Measured per decode
    // step of the 24-layer model against the tcgen05 kernel: 1036 / 1094 / 1129 / 1160 us against 1002 / 1103 / 1160 /
    // 1200 at 33 / 48 / 56 / 64 rows, hence not between 33 and 40.)
    const int splits_wide = std::max((k_blocks + 3) / 4, splits / 2);
    const bool gemv = MODE != sg::B_PLANES && dec->use_gemv && rows_ub <= dec->gemv_rows && !(rows_ub > 32 && rows_ub <= 40) &&
                      (rows_ub <= 32 ? kb_max <= sv::kSvMaxKb : (k_blocks + splits_wide - 1) / splits_wide <= 4);
    ProfScope ps(dec, family + KF_COUNT * (!gemv ? KV_TCGEN05 : rows_ub <= dec->gemv_direct_rows ? KV_GEMV : KV_GEMV_STAGED));
    if constexpr (MODE != sg::B_PLANES) {
        // Steps of at most 32 rows whose CTAs cover at most two k-blocks: warp-level MMAs (step_gemv.cuh), activation
        // fragments straight from global memory up to 8 rows, through shared memory beyond
        if (gemv) {
            cudaLaunchConfig_t gc = {};
            gc.gridDim = dim3(m_tiles, splits, 1);
            gc.blockDim = dim3(sv::kSvThreads);
            const bool direct = rows_ub <= dec->gemv_direct_rows, wide = rows_ub > 32;
            const int nt = rows_ub <= 16 ? 2 : 4;
            if (wide) gc.gridDim = dim3(m_tiles, splits_wide, 2);
            gc.dynamicSmemBytes = direct ? (size_t)sv::kSvMaxKb * tc::kATileBytes + 1024 : (size_t)sv::sv_staged_smem(nt, wide ? 4 : sv::kSvMaxKb);
            gc.stream = dec->stream;
            cudaLaunchAttribute ga[1];
            ga[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            ga[0].val.programmaticStreamSerializationAllowed = dec->use_pdl ? 1 : 0;
            gc.attrs = ga;
            gc.numAttrs = 1;
            const CUtensorMap &second = map_w2 ? *map_w2 : map_w;
            cudaError_t ge = direct    ? cudaLaunchKernelEx(&gc, sv::step_gemv_kernel<MODE, 1>, map_w, second, p)
                             : wide    ? cudaLaunchKernelEx(&gc, sv::step_gemv_staged_kernel<MODE, 4, 4>, map_w, second, p)
                             : nt == 2 ? cudaLaunchKernelEx(&gc, sv::step_gemv_staged_kernel<MODE, 2>, map_w, second, p)
                                       : cudaLaunchKernelEx(&gc, sv::step_gemv_staged_kernel<MODE, 4>, map_w, second, p);
            if (ge != cudaSuccess) return fail(dec, AED_ERR_CUDA, "projection launch: %s", cudaGetErrorString(ge));
            AED_LAUNCHED(dec);
            return AED_OK;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(m_tiles, splits, row_tiles);
    cfg.blockDim = dim3(sg::kSgThreads);
    cfg.dynamicSmemBytes = (size_t)stages * stage_bytes + 1024;
    cfg.stream = dec->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = dec->use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // the accumulator is transposed through the ring's memory before it leaves: n_tile rows of 132 floats
    if (MODE == sg::B_PLANES && (size_t)stages * stage_bytes < (size_t)n_tile * (tc::kTileM + 4) * 4)
        cfg.dynamicSmemBytes = (size_t)n_tile * (tc::kTileM + 4) * 4 + 1024;
    cudaError_t e = MODE == sg::B_PLANES
                        ? cudaLaunchKernelEx(&cfg, sg::step_gemm_kernel<MODE>, map_w, plane_maps[ni][0], plane_maps[ni][1], p)
                        : cudaLaunchKernelEx(&cfg, sg::step_gemm_kernel<MODE>, map_w, src_maps[ni], map_w2 ? *map_w2 : src_maps[ni], p);
    if (e != cudaSuccess) return fail(dec, AED_ERR_CUDA, "projection launch: %s", cudaGetErrorString(e));
    AED_LAUNCHED(dec);
    return AED_OK;
}

// A prefill pass (several prompt positions per utterance, rows = (utterance, position) pairs): the row table and the
// rows' tokens are already in place; keys and values are appended by a kernel of their own before any row attends; only
// the last chunk projects to the vocabulary, and only for the rows of the last position (rows 0 .. batch - 1).
struct PrefillPass { bool last_chunk; int batch; };

aed_status_t forward_step_fused(aed_dec *dec, int rows_ub, int self_len_ub, const int32_t *tokens, float *logits_out,
                                const PrefillPass *pf = nullptr)
{
    typedef __nv_bfloat16 T;
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    const int d = c.d_model, F = c.d_ffn, V = c.vocab;
    float *x = dec->at<float>(L.x), *qkv = dec->at<float>(L.qkv), *hid = dec->at<float>(L.hid), *att = dec->at<float>(L.act);
    float *qc = dec->at<float>(L.qc);
    float2 *stats = dec->at<float2>(L.ln_stats);
    const int stats_stride = rows_bucket(c.max_batch);
    const int32_t *active_list = dec->at<int32_t>(L.active_list), *t_u = dec->at<int32_t>(L.t_u);
    {
        ProfScope ps(dec, KF_EMBED);
        if (pf)
            embed_rows_kernel<T><<<rows_ub, 256, 0, dec->stream>>>(dec->state(), dec->at<int4>(L.row_info), dec->at<int32_t>(L.row_tok),
                                                                   (const T *)dec->embed, dec->at<float>(L.pe), d, V, sqrtf((float)d), x, qkv, 3 * d,
                                                                   qc, d);
        else {
            // starts while the row compaction still runs and waits for it inside (programmatic launch)
            const DecState *state = dec->state();
            const T *emb = (const T *)dec->embed;
            const float *pe = dec->at<float>(L.pe);
            int dd = d, vv = V, zc = 3 * d, zc2 = d;
            float sc = sqrtf((float)d);
            float *zb = qkv, *zb2 = qc;
            void *args[] = {&state, &active_list, &tokens, &t_u, &emb, &pe, &dd, &vv, &sc, &x, &zb, &zc, &zb2, &zc2};
            AED_TRY(launch_pdl_impl(dec, (const void *)embed_kernel<T>, dim3(rows_ub), dim3(256), 0, args));
        }
        if (pf) AED_LAUNCHED(dec);
    }
    const bool pdl = dec->use_pdl;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = dec->layers[l];
        const aed_dec::TcLayerMaps &m = dec->tc_layers[l];
        T *self_cache = dec->at<T>(L.self_cache) + (size_t)l * L.self_layer_elems;
        const T *cross = dec->at<T>(L.cross_store) + (size_t)l * L.cross_layer_elems;
        const float *fc = dec->at<float>(L.fold_c) + (size_t)l * L.fold_layer_floats;
        const float *c1_qkv = fc, *c2_qkv = fc + 3 * d, *c1_qc = fc + 6 * d, *c2_qc = fc + 7 * d, *c1_ff = fc + 8 * d,
                    *c2_ff = fc + 8 * d + F;
        const LayerWeights &wn = dec->layers[(l + 1) % c.n_layers];     // next layer (or layer 0 of the next step)
        const size_t e2 = sizeof(T);
        sg::StepGemmParams p{};
        // 1. [q | k | v] raw = (gamma1 * x) Wqkv^T, and the part of the cross-attention query that this layer's input
        //    already fixes, q'A raw = (gamma2 * x) Wqc^T (the rest follows in 3) ; side: LN1 statistics of x
        p.src = x; p.ld_src = d; p.gamma = (const T *)w.ln1_g;
        p.out = qkv; p.ldo = 3 * d; p.bias = nullptr;
        p.gamma2 = (const T *)w.ln2_g; p.out2 = qc; p.ldo2 = d; p.bias2 = nullptr;
        p.stats_src = x; p.stats_out = stats; p.stats_d = d;
        p.prefetch_ptr = wn.w_qkv; p.prefetch_bytes = (size_t)3 * d * d * e2;
        p.prefetch2_ptr = wn.w_q_c; p.prefetch2_bytes = (size_t)d * d * e2;
        // the vocabulary matrix is as large as a layer: its way into L2 starts a whole layer ahead of the projection
        if (l == c.n_layers - 1) { p.prefetch2_ptr = dec->w_out; p.prefetch2_bytes = (size_t)V * d * e2; }
        AED_TRY(launch_step_gemm<sg::B_GAMMA>(dec, KF_GEMM_QKV, m.qkv, dec->tc_src_x, 3 * d, d, rows_ub, p, nullptr, &m.qc, d));
        // 2. self-attention (applies LN1 to q, k, v; appends k, v)
        if (pf) {
            {
                ProfScope ps(dec, KF_ATTN_SELF);
                const DecState *state = dec->state();
                const int4 *ri = dec->at<int4>(L.row_info);
                const float *qp = qkv;
                int ldq = 3 * d, heads = c.n_heads, cap = c.max_dec_len;
                const float2 *stp = stats;
                void *args[] = {&state, &ri, &qp, &ldq, &self_cache, &heads, &cap, &stp, &c1_qkv, &c2_qkv};
                AED_TRY(launch_pdl_impl(dec, (const void *)append_kv_kernel<T>, dim3(rows_ub, c.n_heads), dim3(kHeadDim), 0, args));
            }
            AED_TRY((launch_attention_fused<T, false, false>(dec, rows_ub, self_len_ub, qkv, 3 * d, self_cache, c.max_dec_len, att,
                                                             nullptr, nullptr, stats, c1_qkv, c2_qkv, pdl)));
        } else {
            AED_TRY((launch_attention_fused<T, false, true>(dec, rows_ub, self_len_ub, qkv, 3 * d, self_cache, c.max_dec_len, att,
                                                            nullptr, nullptr, stats, c1_qkv, c2_qkv, pdl)));
        }
        // 3. x += att Wo^T + bo, and in the same launch the rest of the cross-attention query:
        //    (gamma2 * x_new) Wqc^T = q'A + att (Wqc diag(gamma2) Wo)^T + Wqc (gamma2 * bo), so the query projection does
        //    not wait for the sum over all features of x_new ; side: clear the FFN hidden rows
        p = sg::StepGemmParams{};
        p.src = att; p.ld_src = d;
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_o;
        p.out2 = qc; p.ldo2 = d; p.bias2 = dec->at<float>(L.comp_b) + (size_t)l * d;
        p.zero_buf = hid; p.zero_cols = F;
        p.prefetch_ptr = wn.w_o; p.prefetch_bytes = (size_t)d * d * e2;
        p.prefetch2_ptr = dec->at<T>(L.comp_w) + (size_t)((l + 1) % c.n_layers) * d * d; p.prefetch2_bytes = (size_t)d * d * e2;
        AED_TRY(launch_step_gemm<sg::B_PLAIN>(dec, KF_GEMM_O, m.o, dec->tc_src_att, d, d, rows_ub, p, nullptr, &m.o_qc, d));
        // 4. cross-attention; every block computes the LN2 statistics of its row of x_new itself
        if (c.cross_kv_format == AED_CROSS_KV_E4M3) {
            const fp8e4m3 *cross8 = dec->at<fp8e4m3>(L.cross_store) + (size_t)l * L.cross_layer_elems;
            AED_TRY((launch_attention_fused<fp8e4m3, true, false>(dec, rows_ub, c.max_enc_len, qc, d, cross8, c.max_total_enc_frames, att,
                                                                  nullptr, nullptr, nullptr, c1_qc, c2_qc, pdl, x)));
        } else {
            AED_TRY((launch_attention_fused<T, true, false>(dec, rows_ub, c.max_enc_len, qc, d, cross, c.max_total_enc_frames, att,
                                                            nullptr, nullptr, nullptr, c1_qc, c2_qc, pdl, x)));
        }
        // 5. x += att Woc^T + boc ; side: clear the [q | k | v] rows for the next layer
        p = sg::StepGemmParams{};
        p.src = att; p.ld_src = d;
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_o_c;
        p.zero_buf = qkv; p.zero_cols = 3 * d;
        p.prefetch_ptr = wn.w_o_c; p.prefetch_bytes = (size_t)d * d * e2;
        AED_TRY(launch_step_gemm<sg::B_PLAIN>(dec, KF_GEMM_OC, m.oc, dec->tc_src_att, d, d, rows_ub, p));
        // 6. hidden raw = (gamma3 * x) W1^T ; side: LN3 statistics
        p = sg::StepGemmParams{};
        p.src = x; p.ld_src = d; p.gamma = (const T *)w.ln3_g;
        p.out = hid; p.ldo = F;
        p.stats_src = x; p.stats_out = stats + 2 * stats_stride; p.stats_d = d;
        p.prefetch_ptr = wn.w_ff1; p.prefetch_bytes = (size_t)F * d * e2;
        AED_TRY(launch_step_gemm<sg::B_GAMMA>(dec, KF_GEMM_FF1, m.ff1, dec->tc_src_x, F, d, rows_ub, p));
        // 7. x += relu(LN3-corrected hidden) W2^T + b2 ; side: clear the cross-query rows
        p = sg::StepGemmParams{};
        p.src = hid; p.ld_src = F; p.c1 = c1_ff; p.c2 = c2_ff; p.stats_in = stats + 2 * stats_stride;
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_ff2;
        p.zero_buf = qc; p.zero_cols = d;          // the next layer's first launch accumulates into it
        p.prefetch_ptr = wn.w_ff2; p.prefetch_bytes = (size_t)F * d * e2;
        AED_TRY(launch_step_gemm<sg::B_LN_RELU>(dec, KF_GEMM_FF2, m.ff2, dec->tc_src_hid, d, F, rows_ub, p));
    }
    if (pf && !pf->last_chunk) return AED_OK;
    if (!pf && dec->use_gemv && rows_ub <= vg::kVgRows && d % 128 == 0 && vg::vg_smem(d) <= 227 * 1024) {
        // at most 16 rows: final LayerNorm, vocabulary projection and argmax keys in one kernel (vocab_gemv.cuh)
        ProfScope ps(dec, KF_GEMM_VOCAB + KF_COUNT * KV_GEMV);
        vg::VocabGemvParams vp{};
        vp.vocab = V; vp.d_model = d;
        vp.x = x; vp.gamma = (const T *)dec->final_ln_g;
        vp.c1 = dec->at<float>(L.fold_out); vp.c2 = vp.c1 + V;
        vp.eps = c.ln_eps;
        vp.logits_out = logits_out;
        vp.keys = dec->at<unsigned long long>(L.keys);
        vp.active_list = active_list;
        vp.state = dec->state();
        void *args[] = {(void *)&dec->tc_w_out, &vp};
        return launch_pdl_impl(dec, (const void *)vg::vocab_gemv_kernel, dim3((V + tc::kTileM - 1) / tc::kTileM), dim3(vg::kVgThreads),
                               (size_t)vg::vg_smem(d), args);
    }
    AED_TRY(launch_ln_planes(dec, rows_ub, x, dec->final_ln_g, dec->final_ln_b, nullptr, 0));
    tc::TcParams tp{};
    tp.bias = (const T *)dec->b_out;
    tp.logits_out = logits_out;
    tp.keys = dec->at<unsigned long long>(L.keys);
    tp.active_list = active_list;
    AED_TRY(launch_vocab_gemm(dec, pf ? pf->batch : rows_ub, tp, pf ? pf->batch : -1));
    return AED_OK;
}

// ---- steps with many rows (bf16 mode): activation planes made once per projection input, 12 kernels per layer -------
// With hundreds of rows every feature tile of the fused projections would convert the same activation rows again
// (24 times for the QKV projection) and that conversion, not the tensor cores, would set the pace.  Here a small kernel
// writes gamma * x (with the row statistics) or the ReLU of the corrected hidden layer as bf16 planes once, attention
// writes its output as planes, and the projections fetch both operands by TMA.

template <typename K, typename... Args>
aed_status_t launch_pdl(aed_dec *dec, K kernel, dim3 grid, dim3 block, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = dec->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = dec->use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...);
    if (e != cudaSuccess) return fail(dec, AED_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
    AED_LAUNCHED(dec);
    return AED_OK;
}

aed_status_t forward_step_planes(aed_dec *dec, int rows_ub, int self_len_ub, const int32_t *tokens, float *logits_out)
{
    typedef __nv_bfloat16 T;
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    const int d = c.d_model, F = c.d_ffn, V = c.vocab;
    float *x = dec->at<float>(L.x), *qkv = dec->at<float>(L.qkv), *hid = dec->at<float>(L.hid), *qc = dec->at<float>(L.qc);
    T *ad_hi = dec->at<T>(L.actd_hi), *ad_lo = dec->at<T>(L.actd_lo), *af_hi = dec->at<T>(L.actf_hi), *af_lo = dec->at<T>(L.actf_lo);
    float2 *stats = dec->at<float2>(L.ln_stats);
    const int stats_stride = rows_bucket(c.max_batch);
    const int32_t *active_list = dec->at<int32_t>(L.active_list), *t_u = dec->at<int32_t>(L.t_u);
    {
        ProfScope ps(dec, KF_EMBED);
        embed_kernel<T><<<rows_ub, 256, 0, dec->stream>>>(dec->state(), active_list, tokens, t_u, (const T *)dec->embed,
                                                          dec->at<float>(L.pe), d, V, sqrtf((float)d), x, qkv, 3 * d);
        AED_LAUNCHED(dec);
    }
    const bool pdl = dec->use_pdl;
    const dim3 ln_block(d <= 2048 ? 256 : 1024);
    auto gamma_planes = [&](const void *g, float2 *st, float *zero_buf, int zero_cols) -> aed_status_t {
        ProfScope ps(dec, KF_LAYERNORM);
        return launch_pdl(dec, gamma_planes_kernel<8>, dim3(rows_ub), ln_block, (const DecState *)dec->state(), (const float *)x,
                          (const T *)g, d, c.ln_eps, st, ad_hi, ad_lo, zero_buf, zero_cols);
    };
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = dec->layers[l];
        const aed_dec::TcLayerMaps &m = dec->tc_layers[l];
        T *self_cache = dec->at<T>(L.self_cache) + (size_t)l * L.self_layer_elems;
        const T *cross = dec->at<T>(L.cross_store) + (size_t)l * L.cross_layer_elems;
        const float *fc = dec->at<float>(L.fold_c) + (size_t)l * L.fold_layer_floats;
        const float *c1_qkv = fc, *c2_qkv = fc + 3 * d, *c1_qc = fc + 6 * d, *c2_qc = fc + 7 * d, *c1_ff = fc + 8 * d,
                    *c2_ff = fc + 8 * d + F;
        sg::StepGemmParams p{};
        // self-attention block
        AED_TRY(gamma_planes(w.ln1_g, stats, qc, d));
        p.out = qkv; p.ldo = 3 * d;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_QKV, m.qkv, nullptr, 3 * d, d, rows_ub, p, dec->tc_actd));
        AED_TRY((launch_attention_fused<T, false, true>(dec, rows_ub, self_len_ub, qkv, 3 * d, self_cache, c.max_dec_len, nullptr,
                                                        ad_hi, ad_lo, stats, c1_qkv, c2_qkv, pdl)));
        p = sg::StepGemmParams{};
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_o;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_O, m.o, nullptr, d, d, rows_ub, p, dec->tc_actd));
        // cross-attention block
        AED_TRY(gamma_planes(w.ln2_g, stats + stats_stride, hid, F));
        p = sg::StepGemmParams{};
        p.out = qc; p.ldo = d;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_QC, m.qc, nullptr, d, d, rows_ub, p, dec->tc_actd));
        if (c.cross_kv_format == AED_CROSS_KV_E4M3) {
            const fp8e4m3 *cross8 = dec->at<fp8e4m3>(L.cross_store) + (size_t)l * L.cross_layer_elems;
            AED_TRY((launch_attention_fused<fp8e4m3, true, false>(dec, rows_ub, c.max_enc_len, qc, d, cross8, c.max_total_enc_frames, nullptr,
                                                                  ad_hi, ad_lo, stats + stats_stride, c1_qc, c2_qc, pdl)));
        } else {
            AED_TRY((launch_attention_fused<T, true, false>(dec, rows_ub, c.max_enc_len, qc, d, cross, c.max_total_enc_frames, nullptr,
                                                            ad_hi, ad_lo, stats + stats_stride, c1_qc, c2_qc, pdl)));
        }
        p = sg::StepGemmParams{};
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_o_c;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_OC, m.oc, nullptr, d, d, rows_ub, p, dec->tc_actd));
        // feed-forward block
        AED_TRY(gamma_planes(w.ln3_g, stats + 2 * stats_stride, qkv, 3 * d));
        p = sg::StepGemmParams{};
        p.out = hid; p.ldo = F;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_FF1, m.ff1, nullptr, F, d, rows_ub, p, dec->tc_actd));
        {
            ProfScope ps(dec, KF_LAYERNORM);
            AED_TRY(launch_pdl(dec, lnrelu_planes_kernel, dim3((F / 4 + 255) / 256, rows_ub), dim3(256), (const DecState *)dec->state(),
                               (const float *)hid, F, (const float2 *)(stats + 2 * stats_stride), c1_ff, c2_ff, af_hi, af_lo));
        }
        p = sg::StepGemmParams{};
        p.out = x; p.ldo = d; p.bias = (const T *)w.b_ff2;
        AED_TRY(launch_step_gemm<sg::B_PLANES>(dec, KF_GEMM_FF2, m.ff2, nullptr, d, F, rows_ub, p, dec->tc_actf));
    }
    AED_TRY(launch_ln_planes(dec, rows_ub, x, dec->final_ln_g, dec->final_ln_b, nullptr, 0));
    tc::TcParams tp{};
    tp.bias = (const T *)dec->b_out;
    tp.logits_out = logits_out;
    tp.keys = dec->at<unsigned long long>(L.keys);
    tp.active_list = active_list;
    AED_TRY(launch_vocab_gemm(dec, rows_ub, tp));
    return AED_OK;
}

// Cross K/V of every layer on tensor cores, one persistent launch: D[frame, feature] = enc[frame, :] . w_kv_c[feature, :]
// Cross-K/V of runs of encoder frames: run i is rows src0[i] .. src0[i] + frames[i] - 1 of the tensor at enc_base
// (enc_rows rows in all) and goes to store rows dst0[i] .. (see ckv::CkvSegs; tile0 is filled here).
aed_status_t precompute_tc(aed_dec *dec, const void *enc_base, long long enc_rows, ckv::CkvSegs segs)
{
    typedef __nv_bfloat16 T;
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    if (reinterpret_cast<uintptr_t>(enc_base) % 16) return fail(dec, AED_ERR_INVALID_ARG, "the encoder states must be 16-byte aligned");
    CUtensorMap map_enc;
    if (!encode_map(&map_enc, enc_base, (size_t)enc_rows, c.d_enc, tc::kTileM))
        return fail(dec, AED_ERR_CUDA, "cuTensorMapEncodeTiled failed for the encoder states");
    segs.tile0[0] = 0;
    for (int i = 0; i < segs.n; ++i) segs.tile0[i + 1] = segs.tile0[i] + (segs.frames[i] + tc::kTileM - 1) / tc::kTileM;
    ckv::CkvParams p{};
    p.segs = segs;
    p.frame_capacity = c.max_total_enc_frames;
    p.d_model = c.d_model; p.n_heads = c.n_heads; p.d_enc = c.d_enc;
    p.n_layers = c.n_layers;
    p.store = dec->ws + L.cross_store;
    p.layer_elems = L.cross_layer_elems;
    p.bias = dec->at<const T *>(L.ckv_bias);
    p.state = dec->state();
    const long long tiles = (long long)segs.tile0[segs.n] * c.n_layers * ((2 * c.d_model + ckv::kTileN - 1) / ckv::kTileN);
    ProfScope ps(dec, KF_PRECOMPUTE);
    const unsigned grid = (unsigned)std::min<long long>(tiles, dec->sm_count);
    const size_t smem = ckv::kStages * ckv::kStageBytes + 1024;
    if (c.cross_kv_format == AED_CROSS_KV_E4M3)
        ckv::crosskv_gemm_kernel<true><<<grid, ckv::kCkvThreads, smem, dec->stream>>>(map_enc, dec->at<CUtensorMap>(L.ckv_maps), p);
    else
        ckv::crosskv_gemm_kernel<false><<<grid, ckv::kCkvThreads, smem, dec->stream>>>(map_enc, dec->at<CUtensorMap>(L.ckv_maps), p);
    AED_LAUNCHED(dec);
    return AED_OK;
}

ckv::CkvSegs one_run(int frames, int dst0)
{
    ckv::CkvSegs g{};
    g.n = 1;
    g.src0[0] = 0; g.frames[0] = frames; g.dst0[0] = dst0;
    return g;
}

template <typename T>
aed_status_t precompute_impl(aed_dec *dec, const void *enc_packed, int frames, int frame0)
{
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    GemmEpilogueArgs<T> ep{};
    ep.d_model = c.d_model;
    ep.n_heads = c.n_heads;
    ep.frame_capacity = c.max_total_enc_frames;
    ep.frame0 = frame0;
    for (int l = 0; l < c.n_layers; ++l) {
        ep.cross_store = dec->at<T>(L.cross_store) + (size_t)l * L.cross_layer_elems;
        AED_TRY((launch_gemm<T, T, EPI_CROSSKV>(dec, KF_PRECOMPUTE, frames, frames, (const T *)enc_packed, c.d_enc,
                                                dec->layers[l].w_kv_c, dec->layers[l].b_kv_c, 2 * c.d_model, c.d_enc, ep)));
    }
    return AED_OK;
}

aed_status_t launch_build_active(aed_dec *dec, const uint8_t *mask)
{
    const Layout &L = dec->lay;
    ProfScope ps(dec, KF_BOOKKEEPING);
    build_active_kernel<<<1, 1024, 0, dec->stream>>>(mask, dec->at<int32_t>(L.retired),
                                                     dec->at<int32_t>(L.t_u), dec->cfg.max_dec_len,
                                                     dec->at<int32_t>(L.active_list), dec->state(),
                                                     dec->at<int32_t>(L.enc_len), dec->at<int32_t>(L.enc_off),
                                                     dec->at<int4>(L.row_info), rows_bucket(dec->cfg.max_batch),
                                                     dec->at<int32_t>(L.len_order));
    AED_LAUNCHED(dec);
    return AED_OK;
}

aed_status_t launch_finish(aed_dec *dec, int rows_ub, int32_t *next_out, int greedy, int32_t *tokens_out,
                           int32_t *out_lens)
{
    const Layout &L = dec->lay;
    ProfScope ps(dec, KF_BOOKKEEPING);
    DecState *state = dec->state();
    const int32_t *active_list = dec->at<int32_t>(L.active_list);
    unsigned long long *keys = dec->at<unsigned long long>(L.keys);
    int32_t *t_u = dec->at<int32_t>(L.t_u), *cur_tok = dec->at<int32_t>(L.cur_tok), *retired = dec->at<int32_t>(L.retired);
    const int32_t *max_len = dec->at<int32_t>(L.max_len);
    int eos = dec->cfg.eos_id, ld = dec->cfg.max_dec_len;
    void *args[] = {&state, &active_list, &keys, &t_u, &next_out, &greedy, &cur_tok, &retired, &max_len, &eos, &tokens_out, &ld, &out_lens};
    return launch_pdl_impl(dec, (const void *)finish_step_kernel, dim3((rows_ub + 127) / 128), dim3(128), 0, args);
}

aed_status_t fill_i32(aed_dec *dec, int32_t *p, int32_t v, size_t n)
{
    if (n == 0) return AED_OK;
    ProfScope ps(dec, KF_BOOKKEEPING);
    fill_i32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, dec->stream>>>(p, v, n);
    AED_LAUNCHED(dec);
    return AED_OK;
}

}  // namespace

// ---- C ABI -------------------------------------------------------------------------------------------------

extern "C" size_t aed_dec_workspace_bytes(const aed_dec_config_t *config)
{
    if (!config || !config_supported(*config, nullptr) || !shape_supported(*config, nullptr)) return 0;
    return make_layout(*config).total;
}

extern "C" aed_status_t aed_dec_create(const aed_dec_config_t *config, const aed_dec_weights_t *w, aed_dec_t **out)
{
    if (out) *out = nullptr;
    if (!config || !w || !out) return fail(nullptr, AED_ERR_INVALID_ARG, "config, weights and out must not be NULL");
    std::string why;
    if (!config_supported(*config, &why)) return fail(nullptr, AED_ERR_INVALID_ARG, "%s", why.c_str());
    if (!shape_supported(*config, &why)) return fail(nullptr, AED_ERR_UNSUPPORTED, "%s", why.c_str());
    Layout lay = make_layout(*config);
    if (!config->workspace) return fail(nullptr, AED_ERR_INVALID_ARG, "workspace is NULL");
    if (reinterpret_cast<uintptr_t>(config->workspace) % 256) return fail(nullptr, AED_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    if (config->workspace_bytes < lay.total)
        return fail(nullptr, AED_ERR_CAPACITY, "workspace has %zu bytes, %zu needed", config->workspace_bytes, lay.total);
    const void *const *required[] = {w->ln1_g, w->ln1_b, w->w_qkv, w->w_o, w->ln2_g, w->ln2_b, w->w_q_c, w->w_kv_c,
                                     w->w_o_c, w->ln3_g, w->ln3_b, w->w_ff1, w->w_ff2};
    if (!w->embed || !w->final_ln_g || !w->final_ln_b || !w->w_out)
        return fail(nullptr, AED_ERR_INVALID_ARG, "embed, final_ln_g, final_ln_b and w_out must not be NULL");
    for (auto arr : required) {
        if (!arr) return fail(nullptr, AED_ERR_INVALID_ARG, "a required per-layer weight array is NULL");
        for (int l = 0; l < config->n_layers; ++l)
            if (!arr[l]) return fail(nullptr, AED_ERR_INVALID_ARG, "a required weight of layer %d is NULL", l);
    }
    aed_dec *dec = new (std::nothrow) aed_dec();
    if (!dec) return fail(nullptr, AED_ERR_INVALID_ARG, "out of host memory");
    dec->cfg = *config;
    dec->lay = lay;
    dec->stream = static_cast<cudaStream_t>(config->stream);
    dec->ws = static_cast<char *>(config->workspace);
    dec->embed = w->embed; dec->final_ln_g = w->final_ln_g; dec->final_ln_b = w->final_ln_b;
    dec->w_out = w->w_out; dec->b_out = w->b_out;
    dec->layers.resize(config->n_layers);
    auto opt = [](const void *const *arr, int l) -> const void * { return arr ? arr[l] : nullptr; };
    for (int l = 0; l < config->n_layers; ++l) {
        LayerWeights &lw = dec->layers[l];
        lw.ln1_g = w->ln1_g[l]; lw.ln1_b = w->ln1_b[l]; lw.w_qkv = w->w_qkv[l]; lw.b_qkv = opt(w->b_qkv, l);
        lw.w_o = w->w_o[l]; lw.b_o = opt(w->b_o, l);
        lw.ln2_g = w->ln2_g[l]; lw.ln2_b = w->ln2_b[l]; lw.w_q_c = w->w_q_c[l]; lw.b_q_c = opt(w->b_q_c, l);
        lw.w_kv_c = w->w_kv_c[l]; lw.b_kv_c = opt(w->b_kv_c, l); lw.w_o_c = w->w_o_c[l]; lw.b_o_c = opt(w->b_o_c, l);
        lw.ln3_g = w->ln3_g[l]; lw.ln3_b = w->ln3_b[l]; lw.w_ff1 = w->w_ff1[l]; lw.b_ff1 = opt(w->b_ff1, l);
        lw.w_ff2 = w->w_ff2[l]; lw.b_ff2 = opt(w->b_ff2, l);
    }
    // positional table and zeroed state
    int n = config->max_dec_len * config->d_model;
    fill_pe_kernel<<<(n + 255) / 256, 256, 0, dec->stream>>>(dec->at<float>(lay.pe), config->max_dec_len, config->d_model);
    dec->launches++;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemsetAsync(dec->ws + lay.keys, 0, lay.total - lay.keys, dec->stream);
    if (e != cudaSuccess) {
        aed_status_t s = fail(nullptr, AED_ERR_CUDA, "create: %s", cudaGetErrorString(e));
        delete dec;
        return s;
    }
    {
        const char *no_graph = getenv("AED_DEC_NO_GRAPH");
        dec->use_graphs = !(no_graph && no_graph[0] == '1');
    }
    if (config->dtype == AED_DTYPE_BF16) {
        aed_status_t s = tc_setup(dec);
        if (s != AED_OK) {
            delete dec;
            return s;
        }
    }
    *out = dec;
    return AED_OK;
}

extern "C" aed_status_t aed_dec_precompute_cross_kv(aed_dec_t *dec, const void *enc_packed, const int32_t *enc_lens,
                                                    int32_t batch)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!enc_packed || !enc_lens) return fail(dec, AED_ERR_INVALID_ARG, "enc_packed and enc_lens must not be NULL");
    if (batch < 1) return fail(dec, AED_ERR_INVALID_ARG, "batch must be at least 1");
    if (batch > dec->cfg.max_batch) return fail(dec, AED_ERR_CAPACITY, "batch %d exceeds max_batch %d", batch, dec->cfg.max_batch);
    long long total = 0;
    for (int u = 0; u < batch; ++u) {
        if (enc_lens[u] < 1) return fail(dec, AED_ERR_INVALID_ARG, "enc_lens[%d] = %d: every utterance needs at least one frame", u, enc_lens[u]);
        if (enc_lens[u] > dec->cfg.max_enc_len) return fail(dec, AED_ERR_CAPACITY, "enc_lens[%d] = %d exceeds max_enc_len %d", u, enc_lens[u], dec->cfg.max_enc_len);
        total += enc_lens[u];
    }
    if (total > dec->cfg.max_total_enc_frames)
        return fail(dec, AED_ERR_CAPACITY, "%lld encoder frames exceed max_total_enc_frames %d", total, dec->cfg.max_total_enc_frames);

    const Layout &L = dec->lay;
    std::vector<int32_t> off(batch + 1, 0);
    for (int u = 0; u < batch; ++u) off[u + 1] = off[u] + enc_lens[u];
    // From here on the old batch is gone.
    dec->have_batch = false;
    dec->enc_len.assign(enc_lens, enc_lens + batch);
    dec->enc_off = off;
    dec->batch = batch;
    dec->total_frames = (int)total;
    // Pageable host vectors: cudaMemcpyAsync stages them before returning, so the vectors may change afterwards.
    AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.enc_off, dec->enc_off.data(), (batch + 1) * 4, cudaMemcpyHostToDevice, dec->stream));
    AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.enc_len, dec->enc_len.data(), batch * 4, cudaMemcpyHostToDevice, dec->stream));
    {
        // visiting order of the row compaction: longest encoder output first (ties by utterance index)
        std::vector<int32_t> order(batch);
        for (int u = 0; u < batch; ++u) order[u] = u;
        std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return enc_lens[a] > enc_lens[b]; });
        AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.len_order, order.data(), batch * 4, cudaMemcpyHostToDevice, dec->stream));
    }
    AED_CUDA(dec, cudaMemsetAsync(dec->ws + L.keys, 0, L.enc_off - L.keys, dec->stream));   // keys, state, t_u, retired, lists
    AED_CUDA(dec, cudaMemcpyAsync(&dec->state()->batch, &dec->batch, sizeof(int32_t), cudaMemcpyHostToDevice, dec->stream));
    dec->slot_mode = false;
    aed_status_t s = dec->use_tc ? precompute_tc(dec, enc_packed, dec->total_frames, one_run(dec->total_frames, 0))
                                 : precompute_impl<float>(dec, enc_packed, dec->total_frames, 0);
    if (s != AED_OK) return s;
    dec->have_batch = true;
    dec->fresh_batch = true;
    dec->steps_issued = 0;
    dec->full_steps = 0;
    return AED_OK;
}

extern "C" aed_status_t aed_dec_step(aed_dec_t *dec, const int32_t *tokens_in, const uint8_t *active, float *logits_out,
                                     int32_t *next_out)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!tokens_in) return fail(dec, AED_ERR_INVALID_ARG, "tokens_in must not be NULL");
    if (!dec->have_batch) return fail(dec, AED_ERR_STATE, "aed_dec_step needs a batch: call aed_dec_precompute_cross_kv first");
    if (dec->slot_mode) return fail(dec, AED_ERR_STATE, "aed_dec_step does not run on slots: use aed_dec_greedy_steps");
    if (dec->full_steps >= dec->cfg.max_dec_len)
        return fail(dec, AED_ERR_CAPACITY, "every utterance already holds max_dec_len = %d tokens", dec->cfg.max_dec_len);
    AED_TRY(launch_build_active(dec, active));
    const int rows_ub = dec->batch;
    const int self_len_ub = dec->steps_issued + 1 < dec->cfg.max_dec_len ? dec->steps_issued + 1 : dec->cfg.max_dec_len;
    aed_status_t s = !dec->use_tc ? forward_step<float>(dec, rows_ub, self_len_ub, tokens_in, logits_out)
                     : rows_ub > dec->planes_rows ? forward_step_planes(dec, rows_ub, self_len_ub, tokens_in, logits_out)
                                                  : forward_step_fused(dec, rows_ub, self_len_ub, tokens_in, logits_out);
    if (s != AED_OK) return s;
    AED_TRY(launch_finish(dec, rows_ub, next_out, 0, nullptr, nullptr));
    dec->steps_issued++;
    if (!active) dec->full_steps++;
    dec->fresh_batch = false;
    return AED_OK;
}

// ---- prompt prefill: several positions per utterance in one pass ---------------------------------------------------
extern "C" aed_status_t aed_dec_prefill(aed_dec_t *dec, const int32_t *prompt, int32_t prompt_len, float *logits_out,
                                        int32_t *next_out)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!prompt) return fail(dec, AED_ERR_INVALID_ARG, "prompt must not be NULL");
    if (prompt_len < 1) return fail(dec, AED_ERR_INVALID_ARG, "prompt_len must be at least 1");
    if (!dec->have_batch) return fail(dec, AED_ERR_STATE, "aed_dec_prefill needs a batch: call aed_dec_precompute_cross_kv first");
    if (!dec->fresh_batch) return fail(dec, AED_ERR_STATE, "aed_dec_prefill must directly follow aed_dec_precompute_cross_kv");
    if (prompt_len > dec->cfg.max_dec_len)
        return fail(dec, AED_ERR_CAPACITY, "prompt_len %d exceeds max_dec_len %d", prompt_len, dec->cfg.max_dec_len);
    if (!dec->use_tc) return fail(dec, AED_ERR_UNSUPPORTED, "aed_dec_prefill needs the bf16 configuration (feed the prompt with aed_dec_step in fp32 mode)");
    const Layout &L = dec->lay;
    const int B = dec->batch;
    // (utterance, position) rows share the step's row buffers: max_batch rows per pass
    const int chunk_max = std::max(1, dec->cfg.max_batch / B);
    for (int j0 = 0; j0 < prompt_len; j0 += chunk_max) {
        const int chunk = std::min(chunk_max, prompt_len - j0), rows = B * chunk;
        const bool last = j0 + chunk == prompt_len;
        {
            ProfScope ps(dec, KF_BOOKKEEPING);
            const int slots = rows_bucket(dec->cfg.max_batch);
            build_prefill_rows_kernel<<<(slots + 255) / 256, 256, 0, dec->stream>>>(
                dec->state(), chunk, j0, prompt_len, prompt, dec->at<int32_t>(L.t_u), dec->at<int32_t>(L.enc_len),
                dec->at<int32_t>(L.enc_off), dec->at<int32_t>(L.len_order), dec->at<int32_t>(L.active_list),
                dec->at<int4>(L.row_info), dec->at<int32_t>(L.row_tok), slots);
            AED_LAUNCHED(dec);
        }
        PrefillPass pf{last, B};
        AED_TRY(forward_step_fused(dec, rows, j0 + chunk, nullptr, logits_out, &pf));
        {
            ProfScope ps(dec, KF_BOOKKEEPING);
            DecState *state = dec->state();
            const int32_t *active_list = dec->at<int32_t>(L.active_list);
            unsigned long long *keys = dec->at<unsigned long long>(L.keys);
            int32_t *t_u = dec->at<int32_t>(L.t_u), *cur_tok = dec->at<int32_t>(L.cur_tok);
            int chunk_arg = chunk, last_arg = last ? 1 : 0;
            void *args[] = {&state, &active_list, &keys, &t_u, &chunk_arg, &last_arg, &next_out, &cur_tok};
            AED_TRY(launch_pdl_impl(dec, (const void *)prefill_finish_kernel, dim3((B + 127) / 128), dim3(128), 0, args));
        }
    }
    dec->steps_issued = prompt_len;
    dec->full_steps = prompt_len;
    dec->fresh_batch = false;
    return AED_OK;
}

// ---- step variant for callers that cannot allocate device memory ---------------------------------------------
// The flash-decoding partials (running max, running sum and 64 accumulators per (row, head, chunk)) are the one
// piece of scratch a step needs beyond activations.  This variant keeps them in a fixed array that is part of
// the library image, so a caller that has no allocator at hand can run steps without carving room for them.
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device.  In host code the array's name is only a handle for the
// runtime; the address a kernel can use has to be asked for, once per device, with that device current.
aed_status_t static_scratch_address(aed_dec *dec, float **out)
{
    int dev = -1;
    AED_CUDA(dec, cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(dec, AED_ERR_UNSUPPORTED, "device index %d is out of range", dev);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr)
            return fail(dec, AED_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
        g_static_scratch_addr[dev] = ptr;
    }
    *out = static_cast<float *>(g_static_scratch_addr[dev]);
    return AED_OK;
}
}  // namespace

extern "C" size_t aed_dec_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" aed_status_t aed_dec_step_static_scratch(aed_dec_t *dec, const int32_t *tokens_in, const uint8_t *active,
                                                    float *logits_out, int32_t *next_out)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!dec->have_batch)
        return fail(dec, AED_ERR_STATE, "aed_dec_step_static_scratch needs a batch: call aed_dec_precompute_cross_kv first");
    // Only the fp32 path splits attention over chunks and writes partials; the bf16 step merges inside one block
    // and touches no scratch, so no batch is refused there.
    const size_t need = dec->use_tc ? 0 : (size_t)dec->batch * dec->cfg.n_heads * dec->lay.max_chunks * kPartialStride * sizeof(float);
    if (need > kStaticScratchBytes)
        return fail(dec, AED_ERR_CAPACITY,
                    "batch %d x %d heads x %d chunks needs %zu bytes of attention scratch; the built-in array holds %zu",
                    dec->batch, dec->cfg.n_heads, dec->lay.max_chunks, need, kStaticScratchBytes);
    float *scratch = nullptr;
    AED_TRY(static_scratch_address(dec, &scratch));
    dec->partials_override = scratch;
    aed_status_t s = aed_dec_step(dec, tokens_in, active, logits_out, next_out);
    dec->partials_override = nullptr;
    return s;
}

namespace {

aed_status_t enqueue_greedy_step(aed_dec *dec, int rows_ub, int self_len_ub, int32_t *tokens_out, int32_t *out_lens)
{
    const Layout &L = dec->lay;
    if (self_len_ub > dec->cfg.max_dec_len) self_len_ub = dec->cfg.max_dec_len;
    AED_TRY(launch_build_active(dec, nullptr));
    const int32_t *tok = dec->at<int32_t>(L.cur_tok);
    aed_status_t st = !dec->use_tc ? forward_step<float>(dec, rows_ub, self_len_ub, tok, nullptr)
                      : rows_ub > dec->planes_rows ? forward_step_planes(dec, rows_ub, self_len_ub, tok, nullptr)
                                                   : forward_step_fused(dec, rows_ub, self_len_ub, tok, nullptr);
    if (st != AED_OK) return st;
    return launch_finish(dec, rows_ub, nullptr, 1, tokens_out, out_lens);
}

// Record one greedy step into a graph on the library's capture stream (nothing runs) and instantiate it.
aed_status_t capture_greedy_step(aed_dec *dec, int rows_ub, int self_len_ub, int32_t *tokens_out, int32_t *out_lens,
                                 aed_dec::GraphEntry *entry)
{
    if (!dec->capture_stream)
        AED_CUDA(dec, cudaStreamCreateWithFlags(&dec->capture_stream, cudaStreamNonBlocking));
    cudaStream_t user = dec->stream;
    const int64_t before = dec->launches;
    AED_CUDA(dec, cudaStreamBeginCapture(dec->capture_stream, cudaStreamCaptureModeThreadLocal));
    dec->stream = dec->capture_stream;
    aed_status_t st = enqueue_greedy_step(dec, rows_ub, self_len_ub, tokens_out, out_lens);
    dec->stream = user;
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(dec->capture_stream, &graph);
    entry->nodes = dec->launches - before;
    dec->launches = before;
    if (st != AED_OK) { if (graph) cudaGraphDestroy(graph); return st; }
    if (e != cudaSuccess || !graph) return fail(dec, AED_ERR_CUDA, "cudaStreamEndCapture: %s", cudaGetErrorString(e));
    e = cudaGraphInstantiate(&entry->exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return fail(dec, AED_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e));
    return AED_OK;
}

}  // namespace

extern "C" aed_status_t aed_dec_greedy_decode(aed_dec_t *dec, const int32_t *max_len, int32_t *tokens_out, int32_t *out_lens)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!max_len || !tokens_out || !out_lens) return fail(dec, AED_ERR_INVALID_ARG, "max_len, tokens_out and out_lens must not be NULL");
    if (!dec->have_batch) return fail(dec, AED_ERR_STATE, "aed_dec_greedy_decode needs a batch: call aed_dec_precompute_cross_kv first");
    if (!dec->fresh_batch || dec->slot_mode) return fail(dec, AED_ERR_STATE, "aed_dec_greedy_decode must directly follow aed_dec_precompute_cross_kv");
    const int B = dec->batch;
    int longest = 0;
    for (int u = 0; u < B; ++u) {
        if (max_len[u] < 1) return fail(dec, AED_ERR_INVALID_ARG, "max_len[%d] = %d: must be at least 1", u, max_len[u]);
        if (max_len[u] > dec->cfg.max_dec_len) return fail(dec, AED_ERR_CAPACITY, "max_len[%d] = %d exceeds max_dec_len %d", u, max_len[u], dec->cfg.max_dec_len);
        if (max_len[u] > longest) longest = max_len[u];
    }
    const Layout &L = dec->lay;
    // rows still alive at step s: utterances with max_len > s (exact without EOS, an upper bound with it)
    std::vector<int> alive(longest + 1, 0);
    for (int u = 0; u < B; ++u) alive[max_len[u] - 1]++;
    for (int s = longest - 1; s >= 0; --s) alive[s] += alive[s + 1];

    dec->fresh_batch = false;
    AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.max_len, max_len, B * 4, cudaMemcpyHostToDevice, dec->stream));
    AED_TRY(fill_i32(dec, dec->at<int32_t>(L.cur_tok), dec->cfg.bos_id, B));
    AED_TRY(fill_i32(dec, tokens_out, -1, (size_t)B * dec->cfg.max_dec_len));
    AED_TRY(fill_i32(dec, out_lens, 0, B));
    // With an end-of-sequence id the forced lengths are only upper bounds.  The host then stays at most kWindow steps
    // ahead of the device: before it issues step s it looks at the retired count that step s - kWindow left behind
    // (an asynchronous copy into pinned memory followed by an event) and stops once every utterance has retired.
    const bool probe = dec->cfg.eos_id >= 0;
    constexpr int kWindow = 8;
    if (probe && !dec->probe_host) {
        AED_CUDA(dec, cudaHostAlloc(reinterpret_cast<void **>(&dec->probe_host), aed_dec::kProbeSlots * sizeof(int32_t), cudaHostAllocDefault));
        for (int i = 0; i < aed_dec::kProbeSlots; ++i) AED_CUDA(dec, cudaEventCreateWithFlags(&dec->probe_event[i], cudaEventDisableTiming));
    }
    for (int s = 0; s < longest; ++s) {
        if (probe && s >= kWindow) {
            const int slot = (s - kWindow) % aed_dec::kProbeSlots;
            AED_CUDA(dec, cudaEventSynchronize(dec->probe_event[slot]));
            if (dec->probe_host[slot] >= B) break;           // everything retired kWindow steps ago: the steps in between did nothing
        }
        const int rows_ub = alive[s];
        if (dec->use_graphs && !dec->profiling) {
            // grids are sized for the keyed row count; kernels leave rows beyond the device-side row count alone
            const int rows_b = rows_key(rows_ub), chunks = (s + 1 + kAttnChunk - 1) / kAttnChunk;
            const aed_dec::GraphKey key(rows_b, chunks, tokens_out, out_lens);
            auto it = dec->graphs.find(key);
            if (it == dec->graphs.end()) {
                aed_dec::GraphEntry entry{};
                AED_TRY(capture_greedy_step(dec, rows_b, chunks * kAttnChunk, tokens_out, out_lens, &entry));
                it = dec->graphs.emplace(key, entry).first;
            }
            AED_CUDA(dec, cudaGraphLaunch(it->second.exec, dec->stream));
            dec->launches += it->second.nodes;
        } else {
            AED_TRY(enqueue_greedy_step(dec, rows_ub, s + 1, tokens_out, out_lens));
        }
        dec->steps_issued = s + 1;
        if (probe) {
            const int slot = s % aed_dec::kProbeSlots;
            AED_CUDA(dec, cudaMemcpyAsync(&dec->probe_host[slot], &dec->state()->n_retired, sizeof(int32_t), cudaMemcpyDeviceToHost, dec->stream));
            AED_CUDA(dec, cudaEventRecord(dec->probe_event[slot], dec->stream));
        }
    }
    dec->full_steps = dec->cfg.max_dec_len;   // every utterance is retired: further steps are refused
    return aed_dec_sync_status(dec);
}

// ---- continuous batching: utterances enter and leave slots one by one -----------------------------------------------

extern "C" aed_status_t aed_dec_open_slots(aed_dec_t *dec, int32_t slots)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    const auto &c = dec->cfg;
    if (slots < 1) return fail(dec, AED_ERR_INVALID_ARG, "slots must be at least 1");
    if (slots > c.max_batch) return fail(dec, AED_ERR_CAPACITY, "%d slots exceed max_batch %d", slots, c.max_batch);
    if ((long long)slots * c.max_enc_len > c.max_total_enc_frames)
        return fail(dec, AED_ERR_CAPACITY, "%d slots of max_enc_len %d frames exceed max_total_enc_frames %d", slots, c.max_enc_len,
                    c.max_total_enc_frames);
    const Layout &L = dec->lay;
    dec->have_batch = false;
    dec->batch = slots;
    dec->total_frames = 0;
    dec->enc_len.assign(slots, 0);
    dec->enc_off.assign(slots + 1, 0);
    for (int u = 0; u <= slots; ++u) dec->enc_off[u] = u * c.max_enc_len;       // every slot owns max_enc_len store rows
    dec->slot_t.assign(slots, -1);
    dec->slot_max.assign(slots, 0);
    AED_CUDA(dec, cudaMemsetAsync(dec->ws + L.keys, 0, L.enc_off - L.keys, dec->stream));   // keys, state, t_u, retired, lists
    AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.enc_off, dec->enc_off.data(), (slots + 1) * 4, cudaMemcpyHostToDevice, dec->stream));
    AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.enc_len, dec->enc_len.data(), slots * 4, cudaMemcpyHostToDevice, dec->stream));
    {
        std::vector<int32_t> order(slots);
        for (int u = 0; u < slots; ++u) order[u] = u;
        AED_CUDA(dec, cudaMemcpyAsync(dec->ws + L.len_order, order.data(), slots * 4, cudaMemcpyHostToDevice, dec->stream));
    }
    AED_CUDA(dec, cudaMemcpyAsync(&dec->state()->batch, &dec->batch, sizeof(int32_t), cudaMemcpyHostToDevice, dec->stream));
    AED_TRY(fill_i32(dec, dec->at<int32_t>(L.retired), 1, slots));      // empty slots take no part in a step
    dec->slot_mode = true;
    dec->have_batch = true;
    dec->fresh_batch = false;
    dec->steps_issued = 0;
    dec->full_steps = 0;
    return AED_OK;
}

namespace {

struct Admission { int slot; long long src_row; int frames, max_len; };

aed_status_t check_admission(aed_dec *dec, const Admission &a)
{
    const auto &c = dec->cfg;
    if (a.slot < 0 || a.slot >= dec->batch) return fail(dec, AED_ERR_INVALID_ARG, "slot %d is outside 0..%d", a.slot, dec->batch - 1);
    if (a.frames < 1) return fail(dec, AED_ERR_INVALID_ARG, "enc_len = %d: an utterance needs at least one frame", a.frames);
    if (a.frames > c.max_enc_len) return fail(dec, AED_ERR_CAPACITY, "enc_len = %d exceeds max_enc_len %d", a.frames, c.max_enc_len);
    if (a.max_len < 1) return fail(dec, AED_ERR_INVALID_ARG, "max_len = %d: must be at least 1", a.max_len);
    if (a.max_len > c.max_dec_len) return fail(dec, AED_ERR_CAPACITY, "max_len = %d exceeds max_dec_len %d", a.max_len, c.max_dec_len);
    // Without an end-of-sequence id the host knows when a slot's utterance ends; with one the caller has seen
    // out_lens[slot] > 0 before it reuses the slot.
    if (c.eos_id < 0 && dec->slot_t[a.slot] >= 0 && dec->slot_t[a.slot] < dec->slot_max[a.slot])
        return fail(dec, AED_ERR_STATE, "slot %d still decodes (%d of %d tokens)", a.slot, dec->slot_t[a.slot], dec->slot_max[a.slot]);
    return AED_OK;
}

// Up to ckv::kMaxSegs utterances enter their slots with one cross-K/V launch and one bookkeeping launch.  The encoder
// states of admission i are rows src_row .. src_row + frames - 1 of the tensor at enc_base (enc_rows rows).
aed_status_t admit_many(aed_dec *dec, const void *enc_base, long long enc_rows, const Admission *adm, int n, int32_t *out_lens)
{
    static_assert(kMaxAdmit == ckv::kMaxSegs, "one bookkeeping entry per run of frames");
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    const size_t row_bytes = (size_t)c.d_enc * (c.dtype == AED_DTYPE_BF16 ? 2 : 4);
    ckv::CkvSegs segs{};
    AdmitBatch ab{};
    segs.n = ab.n = n;
    for (int i = 0; i < n; ++i) {
        AED_TRY(check_admission(dec, adm[i]));
        for (int k = 0; k < i; ++k)
            if (adm[k].slot == adm[i].slot) return fail(dec, AED_ERR_INVALID_ARG, "slot %d is admitted into twice", adm[i].slot);
        segs.src0[i] = (int)adm[i].src_row; segs.frames[i] = adm[i].frames; segs.dst0[i] = adm[i].slot * c.max_enc_len;
        ab.slot[i] = adm[i].slot; ab.n_frames[i] = adm[i].frames; ab.frame0[i] = segs.dst0[i]; ab.forced_len[i] = adm[i].max_len;
    }
    if (dec->use_tc) {
        AED_TRY(precompute_tc(dec, enc_base, enc_rows, segs));
    } else {
        for (int i = 0; i < n; ++i)
            AED_TRY(precompute_impl<float>(dec, static_cast<const char *>(enc_base) + (size_t)adm[i].src_row * row_bytes, adm[i].frames, segs.dst0[i]));
    }
    {
        ProfScope ps(dec, KF_BOOKKEEPING);
        admit_slots_kernel<<<1, 32, 0, dec->stream>>>(ab, c.bos_id, dec->at<int32_t>(L.enc_len), dec->at<int32_t>(L.enc_off),
                                                      dec->at<int32_t>(L.t_u), dec->at<int32_t>(L.retired), dec->at<int32_t>(L.cur_tok),
                                                      dec->at<int32_t>(L.max_len), out_lens);
        AED_LAUNCHED(dec);
    }
    for (int i = 0; i < n; ++i) {
        dec->enc_len[adm[i].slot] = adm[i].frames;
        dec->slot_t[adm[i].slot] = 0;
        dec->slot_max[adm[i].slot] = adm[i].max_len;
    }
    return AED_OK;
}

}  // namespace

extern "C" aed_status_t aed_dec_admit(aed_dec_t *dec, int32_t slot, const void *enc, int32_t enc_len, int32_t max_len,
                                      int32_t *out_lens)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!dec->have_batch || !dec->slot_mode) return fail(dec, AED_ERR_STATE, "aed_dec_admit needs slots: call aed_dec_open_slots first");
    if (!enc) return fail(dec, AED_ERR_INVALID_ARG, "enc must not be NULL");
    const Admission a{slot, 0, enc_len, max_len};
    AED_TRY(check_admission(dec, a));           // before enc_len is used as the extent of the tensor
    return admit_many(dec, enc, enc_len, &a, 1, out_lens);
}

extern "C" aed_status_t aed_dec_greedy_steps(aed_dec_t *dec, int32_t n_steps, int32_t *tokens_out, int32_t *out_lens,
                                             int32_t *steps_done)
{
    if (steps_done) *steps_done = 0;
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!dec->have_batch || !dec->slot_mode) return fail(dec, AED_ERR_STATE, "aed_dec_greedy_steps needs slots: call aed_dec_open_slots first");
    if (!tokens_out || !out_lens) return fail(dec, AED_ERR_INVALID_ARG, "tokens_out and out_lens must not be NULL");
    if (n_steps < 0) return fail(dec, AED_ERR_INVALID_ARG, "n_steps must not be negative");
    for (int s = 0; s < n_steps; ++s) {
        // what the host knows: a slot decodes until its forced length (with an end-of-sequence id it may stop earlier
        // on the device; its row then simply is not there any more)
        int rows_ub = 0, longest = 0;
        for (int u = 0; u < dec->batch; ++u)
            if (dec->slot_t[u] >= 0 && dec->slot_t[u] < dec->slot_max[u]) { ++rows_ub; longest = std::max(longest, dec->slot_t[u] + 1); }
        if (rows_ub == 0) break;
        if (dec->use_graphs && !dec->profiling) {
            const int rows_b = rows_key(rows_ub), chunks = (longest + kAttnChunk - 1) / kAttnChunk;
            const aed_dec::GraphKey key(rows_b, chunks, tokens_out, out_lens);
            auto it = dec->graphs.find(key);
            if (it == dec->graphs.end()) {
                aed_dec::GraphEntry entry{};
                AED_TRY(capture_greedy_step(dec, rows_b, chunks * kAttnChunk, tokens_out, out_lens, &entry));
                it = dec->graphs.emplace(key, entry).first;
            }
            AED_CUDA(dec, cudaGraphLaunch(it->second.exec, dec->stream));
            dec->launches += it->second.nodes;
        } else {
            AED_TRY(enqueue_greedy_step(dec, rows_ub, longest, tokens_out, out_lens));
        }
        for (int u = 0; u < dec->batch; ++u)
            if (dec->slot_t[u] >= 0 && dec->slot_t[u] < dec->slot_max[u]) ++dec->slot_t[u];
        if (steps_done) ++*steps_done;
    }
    return AED_OK;
}

extern "C" aed_status_t aed_dec_decode_stream(aed_dec_t *dec, const void *enc_packed, const int32_t *enc_lens,
                                              const int32_t *max_lens, const int32_t *order, int32_t n, int32_t slots,
                                              int32_t poll_steps, int32_t *tokens_out, int32_t *out_lens,
                                              int64_t *steps_out, int64_t *row_steps_out)
{
    if (steps_out) *steps_out = 0;
    if (row_steps_out) *row_steps_out = 0;
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!enc_packed || !enc_lens || !max_lens || !tokens_out || !out_lens)
        return fail(dec, AED_ERR_INVALID_ARG, "enc_packed, enc_lens, max_lens, tokens_out and out_lens must not be NULL");
    if (n < 1) return fail(dec, AED_ERR_INVALID_ARG, "n must be at least 1");
    const auto &c = dec->cfg;
    const bool eos = c.eos_id >= 0;
    if (eos && poll_steps < 1) return fail(dec, AED_ERR_INVALID_ARG, "poll_steps must be at least 1 when eos_id >= 0");
    std::vector<long long> off(n + 1, 0);
    std::vector<char> seen(n, 0);
    for (int i = 0; i < n; ++i) {
        if (enc_lens[i] < 1 || enc_lens[i] > c.max_enc_len)
            return fail(dec, enc_lens[i] < 1 ? AED_ERR_INVALID_ARG : AED_ERR_CAPACITY, "enc_lens[%d] = %d is outside 1..max_enc_len = %d", i, enc_lens[i], c.max_enc_len);
        if (max_lens[i] < 1 || max_lens[i] > c.max_dec_len)
            return fail(dec, max_lens[i] < 1 ? AED_ERR_INVALID_ARG : AED_ERR_CAPACITY, "max_lens[%d] = %d is outside 1..max_dec_len = %d", i, max_lens[i], c.max_dec_len);
        off[i + 1] = off[i] + enc_lens[i];
        if (order) {
            if (order[i] < 0 || order[i] >= n || seen[order[i]]) return fail(dec, AED_ERR_INVALID_ARG, "order is not a permutation of 0..n-1");
            seen[order[i]] = 1;
        }
    }
    AED_TRY(aed_dec_open_slots(dec, slots));
    const Layout &L = dec->lay;
    if (off[n] > 0x7fffffffLL) return fail(dec, AED_ERR_CAPACITY, "the stream has %lld encoder frames; at most 2^31 - 1 per call", off[n]);
    // The scheduling decisions are in stream_schedule.h; here are its operations on the device.
    struct Ops {
        aed_dec *dec;
        const void *enc_packed;
        const std::vector<long long> &off;
        const int32_t *enc_lens, *max_lens;
        int32_t *toks, *lens, *tokens_out, *out_lens;
        int ld, slots;
        int admit(const StreamAdmission *a, int k)
        {
            Admission adm[ckv::kMaxSegs];
            for (int i = 0; i < k; ++i) adm[i] = Admission{a[i].slot, off[a[i].utterance], enc_lens[a[i].utterance], max_lens[a[i].utterance]};
            return admit_many(dec, enc_packed, off.back(), adm, k, lens);
        }
        int steps(int want, int *done)
        {
            int32_t d = 0;
            const aed_status_t st = aed_dec_greedy_steps(dec, want, toks, lens, &d);
            *done = d;
            return st;
        }
        int read_lens(int32_t *host)
        {
            if (cudaMemcpyAsync(host, lens, (size_t)slots * 4, cudaMemcpyDeviceToHost, dec->stream) != cudaSuccess ||
                cudaStreamSynchronize(dec->stream) != cudaSuccess)
                return fail(dec, AED_ERR_CUDA, "reading the slot lengths: %s", cudaGetErrorString(cudaGetLastError()));
            return AED_OK;
        }
        // The finished utterance's tokens and length go to the host behind the steps that produced them and before
        // the slot's next occupant (stream order); with pinned host buffers the host does not wait for them.
        int harvest(int s, int u)
        {
            if (cudaMemcpyAsync(tokens_out + (size_t)u * ld, toks + (size_t)s * ld, (size_t)max_lens[u] * 4, cudaMemcpyDeviceToHost, dec->stream) != cudaSuccess ||
                cudaMemcpyAsync(out_lens + u, lens + s, 4, cudaMemcpyDeviceToHost, dec->stream) != cudaSuccess)
                return fail(dec, AED_ERR_CUDA, "copying a finished utterance out: %s", cudaGetErrorString(cudaGetLastError()));
            return AED_OK;
        }
    } ops{dec, enc_packed, off, enc_lens, max_lens, dec->at<int32_t>(L.slot_tokens), dec->at<int32_t>(L.slot_lens), tokens_out,
          out_lens, c.max_dec_len, slots};
    StreamTotals tot;
    const int rc = run_stream_schedule(n, slots, order, max_lens, eos, poll_steps, ckv::kMaxSegs, ops, &tot);
    if (rc < 0) return static_cast<aed_status_t>(rc);
    const long long steps = tot.steps, row_steps = tot.row_steps;
    if (steps_out) *steps_out = steps;
    if (row_steps_out) *row_steps_out = row_steps;
    return aed_dec_sync_status(dec);
}

extern "C" aed_status_t aed_dec_sync_status(aed_dec_t *dec)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    DecState host{};
    AED_CUDA(dec, cudaMemcpyAsync(&host, dec->state(), sizeof host, cudaMemcpyDeviceToHost, dec->stream));
    AED_CUDA(dec, cudaStreamSynchronize(dec->stream));
    const aed_status_t s = aed_dec_status_of_error_word(host.error);
    if (s == AED_ERR_CAPACITY) return fail(dec, s, "a step was asked of an utterance whose self-attention cache is full");
    if (s != AED_OK) return fail(dec, s, "a bounded wait on the device ran out (device-side error %d)", host.error);
    return AED_OK;
}

// The sticky error word of the device-side decode state as a status: 0 = fine, 1 = a self-attention cache was full,
// anything else = a kernel gave up waiting.
extern "C" aed_status_t aed_dec_status_of_error_word(int32_t error_word)
{
    if (error_word == 0) return AED_OK;
    if (error_word == 1) return AED_ERR_CAPACITY;
    return AED_ERR_TIMEOUT;
}

extern "C" aed_status_t aed_dec_profile_enable(aed_dec_t *dec, int32_t enable)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    AED_CUDA(dec, cudaStreamSynchronize(dec->stream));
    dec->profiling = enable != 0;
    dec->prof_used = 0;
    dec->prof_family.clear();
    return AED_OK;
}

extern "C" int32_t aed_dec_profile_read(aed_dec_t *dec, int32_t max_families, const char **names, double *ms,
                                        int64_t *launches)
{
    if (!dec || !names || !ms || !launches || max_families < 1) return AED_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(dec->stream) != cudaSuccess) return AED_ERR_CUDA;
    double sum[KF_COUNT * KV_COUNT] = {0};
    int64_t cnt[KF_COUNT * KV_COUNT] = {0};
    static std::string variant_names[KF_COUNT * KV_COUNT];
    static std::once_flag once;
    std::call_once(once, [] {
        for (int v = 0; v < KV_COUNT; ++v)
            for (int f = 0; f < KF_COUNT; ++f) variant_names[f + KF_COUNT * v] = std::string(kFamilyNames[f]) + kVariantSuffix[v];
    });
    for (size_t i = 0; i < dec->prof_family.size() && 2 * i + 1 < dec->prof_used + 1; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, dec->prof_events[2 * i], dec->prof_events[2 * i + 1]) != cudaSuccess) continue;
        sum[dec->prof_family[i]] += t;
        cnt[dec->prof_family[i]]++;
    }
    int n = 0;
    for (int f = 0; f < KF_COUNT * KV_COUNT && n < max_families; ++f) {
        if (!cnt[f]) continue;
        names[n] = variant_names[f].c_str(); ms[n] = sum[f]; launches[n] = cnt[f];
        ++n;
    }
    return n;
}

extern "C" int64_t aed_dec_launch_count(const aed_dec_t *dec) { return dec ? dec->launches : 0; }

extern "C" void aed_dec_destroy(aed_dec_t *dec)
{
    if (!dec) return;
    for (cudaEvent_t e : dec->prof_events) cudaEventDestroy(e);
    for (auto &g : dec->graphs) cudaGraphExecDestroy(g.second.exec);
    if (dec->capture_stream) cudaStreamDestroy(dec->capture_stream);
    for (cudaEvent_t e : dec->probe_event) if (e) cudaEventDestroy(e);
    if (dec->probe_host) cudaFreeHost(dec->probe_host);
    delete dec;
}

extern "C" const char *aed_dec_last_error(const aed_dec_t *dec) { return dec ? dec->err.c_str() : ""; }

extern "C" const char *aed_dec_create_error(void) { return g_create_error.c_str(); }
