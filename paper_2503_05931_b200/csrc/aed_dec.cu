// Host side of the AED decoder library: handle, workspace layout, launch sequences, C ABI.
#include "../../include/aed_dec.h"

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "step_kernels.cuh"

using namespace aed;

namespace {

thread_local std::string g_create_error;

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct LayerWeights {
    const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o;
    const void *ln2_g, *ln2_b, *w_q_c, *b_q_c, *w_kv_c, *b_kv_c, *w_o_c, *b_o_c;
    const void *ln3_g, *ln3_b, *w_ff1, *b_ff1, *w_ff2, *b_ff2;
};

// Byte offsets of every region of the caller's workspace.
struct Layout {
    size_t self_cache, cross_store, x, act, qkv, hid, partials, pe, keys, state;
    size_t t_u, retired, active_list, cur_tok, enc_off, enc_len, max_len, total;
    size_t self_layer_elems, cross_layer_elems;
    int max_chunks;
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
    return true;
}

bool shape_supported(const aed_dec_config_t &c, std::string *why)
{
    auto fail = [&](const char *m) { if (why) *why = m; return false; };
    if (c.d_model % c.n_heads != 0 || c.d_model / c.n_heads != kHeadDim) return fail("head_dim must be 64");
    if (c.d_model % 64 || c.d_ffn % 64 || c.d_enc % 64) return fail("d_model, d_ffn and d_enc must be multiples of 64");
    if (c.d_model > 8192) return fail("d_model above 8192 is not supported");
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
    L.cross_store = take(L.cross_layer_elems * c.n_layers * e);
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
    L.t_u = take(B * 4);
    L.retired = take(B * 4);
    L.active_list = take(B * 4);
    L.cur_tok = take(B * 4);
    L.enc_off = take((B + 1) * 4);
    L.enc_len = take(B * 4);
    L.max_len = take(B * 4);
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
    std::string err;
    int64_t launches = 0;
    // optional per-kernel-family timing (CUDA events around every launch)
    bool profiling = false;
    std::vector<cudaEvent_t> prof_events;          // pool, two per recorded launch
    std::vector<int> prof_family;                  // family of each recorded launch
    size_t prof_used = 0;
    // set only while aed_dec_step_static_scratch runs: attention partials go here instead of the workspace
    float *partials_override = nullptr;

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

template <typename T, bool kCross>
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
    attn_partial_kernel<T, kCross><<<grid, 128, 0, dec->stream>>>(
        dec->state(), dec->at<int32_t>(dec->lay.active_list), q, ldq, cache, H, seq_capacity,
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

template <typename T>
aed_status_t precompute_impl(aed_dec *dec, const void *enc_packed)
{
    const auto &c = dec->cfg;
    const Layout &L = dec->lay;
    GemmEpilogueArgs<T> ep{};
    ep.d_model = c.d_model;
    ep.n_heads = c.n_heads;
    ep.frame_capacity = c.max_total_enc_frames;
    for (int l = 0; l < c.n_layers; ++l) {
        ep.cross_store = dec->at<T>(L.cross_store) + (size_t)l * L.cross_layer_elems;
        AED_TRY((launch_gemm<T, T, EPI_CROSSKV>(dec, KF_PRECOMPUTE, dec->total_frames, dec->total_frames, (const T *)enc_packed, c.d_enc,
                                                dec->layers[l].w_kv_c, dec->layers[l].b_kv_c, 2 * c.d_model, c.d_enc, ep)));
    }
    return AED_OK;
}

aed_status_t launch_build_active(aed_dec *dec, const uint8_t *mask)
{
    const Layout &L = dec->lay;
    ProfScope ps(dec, KF_BOOKKEEPING);
    build_active_kernel<<<1, 1024, 0, dec->stream>>>(dec->batch, mask, dec->at<int32_t>(L.retired),
                                                     dec->at<int32_t>(L.t_u), dec->cfg.max_dec_len,
                                                     dec->at<int32_t>(L.active_list), dec->state());
    AED_LAUNCHED(dec);
    return AED_OK;
}

aed_status_t launch_finish(aed_dec *dec, int rows_ub, int32_t *next_out, int greedy, int32_t *tokens_out,
                           int32_t *out_lens)
{
    const Layout &L = dec->lay;
    ProfScope ps(dec, KF_BOOKKEEPING);
    finish_step_kernel<<<(rows_ub + 127) / 128, 128, 0, dec->stream>>>(
        dec->state(), dec->at<int32_t>(L.active_list), dec->at<unsigned long long>(L.keys), dec->at<int32_t>(L.t_u),
        next_out, greedy, dec->at<int32_t>(L.cur_tok), dec->at<int32_t>(L.retired), dec->at<int32_t>(L.max_len),
        dec->cfg.eos_id, tokens_out, dec->cfg.max_dec_len, out_lens);
    AED_LAUNCHED(dec);
    return AED_OK;
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
    AED_CUDA(dec, cudaMemsetAsync(dec->ws + L.keys, 0, L.enc_off - L.keys, dec->stream));   // keys, state, t_u, retired, lists
    aed_status_t s = dec->cfg.dtype == AED_DTYPE_BF16 ? precompute_impl<__nv_bfloat16>(dec, enc_packed)
                                                      : precompute_impl<float>(dec, enc_packed);
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
    if (dec->full_steps >= dec->cfg.max_dec_len)
        return fail(dec, AED_ERR_CAPACITY, "every utterance already holds max_dec_len = %d tokens", dec->cfg.max_dec_len);
    AED_TRY(launch_build_active(dec, active));
    const int rows_ub = dec->batch;
    const int self_len_ub = dec->steps_issued + 1 < dec->cfg.max_dec_len ? dec->steps_issued + 1 : dec->cfg.max_dec_len;
    aed_status_t s = dec->cfg.dtype == AED_DTYPE_BF16
                         ? forward_step<__nv_bfloat16>(dec, rows_ub, self_len_ub, tokens_in, logits_out)
                         : forward_step<float>(dec, rows_ub, self_len_ub, tokens_in, logits_out);
    if (s != AED_OK) return s;
    AED_TRY(launch_finish(dec, rows_ub, next_out, 0, nullptr, nullptr));
    dec->steps_issued++;
    if (!active) dec->full_steps++;
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
    const size_t need = (size_t)dec->batch * dec->cfg.n_heads * dec->lay.max_chunks * kPartialStride * sizeof(float);
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

extern "C" aed_status_t aed_dec_greedy_decode(aed_dec_t *dec, const int32_t *max_len, int32_t *tokens_out, int32_t *out_lens)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (!max_len || !tokens_out || !out_lens) return fail(dec, AED_ERR_INVALID_ARG, "max_len, tokens_out and out_lens must not be NULL");
    if (!dec->have_batch) return fail(dec, AED_ERR_STATE, "aed_dec_greedy_decode needs a batch: call aed_dec_precompute_cross_kv first");
    if (!dec->fresh_batch) return fail(dec, AED_ERR_STATE, "aed_dec_greedy_decode must directly follow aed_dec_precompute_cross_kv");
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
    const bool bf16 = dec->cfg.dtype == AED_DTYPE_BF16;
    for (int s = 0; s < longest; ++s) {
        const int rows_ub = alive[s];
        AED_TRY(launch_build_active(dec, nullptr));
        aed_status_t st = bf16 ? forward_step<__nv_bfloat16>(dec, rows_ub, s + 1, dec->at<int32_t>(L.cur_tok), nullptr)
                               : forward_step<float>(dec, rows_ub, s + 1, dec->at<int32_t>(L.cur_tok), nullptr);
        if (st != AED_OK) return st;
        AED_TRY(launch_finish(dec, rows_ub, nullptr, 1, tokens_out, out_lens));
        dec->steps_issued = s + 1;
    }
    dec->full_steps = dec->cfg.max_dec_len;   // every utterance is retired: further steps are refused
    return aed_dec_sync_status(dec);
}

extern "C" aed_status_t aed_dec_sync_status(aed_dec_t *dec)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    DecState host{};
    AED_CUDA(dec, cudaMemcpyAsync(&host, dec->state(), sizeof host, cudaMemcpyDeviceToHost, dec->stream));
    AED_CUDA(dec, cudaStreamSynchronize(dec->stream));
    if (host.error == 1) return fail(dec, AED_ERR_CAPACITY, "a step was asked of an utterance whose self-attention cache is full");
    if (host.error != 0) return fail(dec, AED_ERR_TIMEOUT, "device-side error %d", host.error);
    return AED_OK;
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
    double sum[KF_COUNT] = {0};
    int64_t cnt[KF_COUNT] = {0};
    for (size_t i = 0; i < dec->prof_family.size() && 2 * i + 1 < dec->prof_used + 1; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, dec->prof_events[2 * i], dec->prof_events[2 * i + 1]) != cudaSuccess) continue;
        sum[dec->prof_family[i]] += t;
        cnt[dec->prof_family[i]]++;
    }
    int n = 0;
    for (int f = 0; f < KF_COUNT && n < max_families; ++f) {
        if (!cnt[f]) continue;
        names[n] = kFamilyNames[f]; ms[n] = sum[f]; launches[n] = cnt[f];
        ++n;
    }
    return n;
}

extern "C" int64_t aed_dec_launch_count(const aed_dec_t *dec) { return dec ? dec->launches : 0; }

extern "C" void aed_dec_destroy(aed_dec_t *dec)
{
    if (!dec) return;
    for (cudaEvent_t e : dec->prof_events) cudaEventDestroy(e);
    delete dec;
}

extern "C" const char *aed_dec_last_error(const aed_dec_t *dec) { return dec ? dec->err.c_str() : ""; }

extern "C" const char *aed_dec_create_error(void) { return g_create_error.c_str(); }
