// Host side of the C ABI declared in include/arl2.h: argument checks, workspace layout,
// kernel selection and launches.  No device memory is allocated here.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "arl2_internal.h"

namespace arl2 {

static thread_local char g_error[512] = "";

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
}

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    size_t status, split_ml, split_o, k_rot, partials, partials_g, state_bf16, state_bf16_b, wq_op, wk_op, wv_op, rope_h, dec_w, dec_total, tok_w, tok_u1, tok_kh, tok_gc, total;
    int nsplit, nchunk, nslot;
};

bool valid_config(const arl2_config* c)
{
    if (c == nullptr) { set_error("config is NULL"); return false; }
    if (c->struct_size != sizeof(arl2_config)) {
        set_error("config.struct_size is %u, this library expects %zu", c->struct_size,
                  sizeof(arl2_config));
        return false;
    }
    if (c->B < 1 || c->H < 1 || c->L < 1) {
        set_error("B, H and L must be >= 1 (got B=%d H=%d L=%d)", c->B, c->H, c->L);
        return false;
    }
    if ((int64_t)c->B * c->H > 65535 * 8 || c->H > 65535 || c->B > 65535) {
        set_error("B=%d, H=%d exceed the launch grid limits", c->B, c->H);
        return false;
    }
    if (c->D != 64 && c->D != 128) { set_error("D must be 64 or 128 (got %d)", c->D); return false; }
    if (c->io_dtype != ARL2_BF16 && c->io_dtype != ARL2_FP32) {
        set_error("io_dtype must be ARL2_BF16 or ARL2_FP32 (got %d)", c->io_dtype);
        return false;
    }
    if ((c->flags & ARL2_FLAG_GATE_SCALAR) && (c->flags & ARL2_FLAG_GATE_ELEMENTWISE)) {
        set_error("ARL2_FLAG_GATE_SCALAR and ARL2_FLAG_GATE_ELEMENTWISE exclude each other");
        return false;
    }
    if (c->commit_rule != 0) {
        set_error("commit_rule %d is reserved; only 0 (gated linear) is built", c->commit_rule);
        return false;
    }
    if (!(c->softmax_scale >= 0.0f) || !(c->l2_eps >= 0.0f) || isinf(c->softmax_scale) ||
        isinf(c->l2_eps)) {
        set_error("softmax_scale and l2_eps must be finite and >= 0");
        return false;
    }
    if ((size_t)c->B * c->L * c->H * c->D >= ((size_t)1 << 40)) {
        set_error("tensor too large");
        return false;
    }
    return true;
}

Layout make_layout(const arl2_config& c)
{
    Layout l;
    size_t esz = c.io_dtype == ARL2_FP32 ? 4 : 2;
    size_t tensor = (size_t)c.B * c.L * c.H * c.D * esz;
    size_t dd = (size_t)c.D * c.D;
    l.nsplit = (c.L + kCommitChunk - 1) / kCommitChunk;
    size_t off = 0;
    l.status = off;     off += align_up(kStatusWords * sizeof(uint32_t));
    // key-range split of the step kernel's last wave (tensor-core path): the parts' row statistics
    // and unnormalised rows
    l.split_ml = l.split_o = off;
    if (tc_supported(c)) {
        l.split_ml = off;      off += align_up((size_t)kSplitTileParts * 128 * 2 * sizeof(float));
        l.split_o = off;       off += align_up((size_t)kSplitTileParts * 128 * 128 * sizeof(float));
    }
    l.k_rot = off;      off += align_up(tensor);
    // partial-sum slots per (stream, head): the plain-FMA kernels use one per 512-token chunk; the
    // tensor-core kernel one per run of tiles a head falls into, runs sized for a 148-SM device
    // (with more SMs the launcher lengthens the runs to fit)
    {
        const long ntile = (c.L + 127) / 128, total = (long)c.B * c.H * ntile;
        long share = (total + 147) / 148;
        if (share < 2) share = 2;
        const long tc_slots = (ntile + share - 1) / share + 1;
        l.nslot = (int)(tc_slots > l.nsplit ? tc_slots : l.nsplit);
    }
    l.partials = off;   off += align_up((size_t)c.B * c.H * l.nslot * dd * sizeof(float));
    l.partials_g = off; off += align_up((size_t)c.B * c.H * l.nslot * dd * sizeof(float));   // delta rule
    // two bf16 operand copies of S: a tensor-core commit writes the one that is not current
    l.state_bf16 = off; off += align_up((size_t)c.B * c.H * dd * 2);
    l.state_bf16_b = off; off += align_up((size_t)c.B * c.H * dd * 2);
    l.wq_op = off;      off += align_up((size_t)c.H * dd * 2);
    l.wk_op = off;      off += align_up((size_t)c.H * dd * 2);
    l.wv_op = off;      off += align_up((size_t)c.H * dd * 2);
    l.rope_h = off;     off += align_up((size_t)((c.L + 127) / 128) * 128 * (c.D / 2) * 4);
    // per-token decay weights of arl2_commit_decay_tokens (small)
    l.dec_w = off;      off += align_up((size_t)c.B * c.L * c.H * sizeof(float));
    l.dec_total = off;  off += align_up((size_t)c.B * c.H * sizeof(float));
    // scratch of arl2_commit_tokens, only when the context asks for it
    l.nchunk = (c.L + kTokenChunk - 1) / kTokenChunk;
    l.tok_w = l.tok_u1 = l.tok_kh = l.tok_gc = 0;
    if (c.flags & ARL2_FLAG_TOKEN_GATES) {
        size_t per = align_up((size_t)c.B * c.H * l.nchunk * kTokenChunk * c.D * sizeof(float));
        l.tok_w = off;  off += per;
        l.tok_u1 = off; off += per;
        l.tok_kh = off; off += per;
        l.tok_gc = off; off += align_up((size_t)c.B * c.H * (l.nchunk + 1) * sizeof(float));   // up to 2 per 128-token tile
    }
    l.total = off;
    return l;
}

}  // namespace
}  // namespace arl2

using namespace arl2;

struct arl2_ctx {
    arl2_config cfg;
    Shape shape;
    Layout lay;
    float* state;
    uint8_t* ws;
    const void *wq, *wk, *wv;
    const float *rope_cos, *rope_sin;
    bool use_tc;
    uint64_t launches;
    uint32_t step_calls;   // parity selects the scheduler counter of the next step launch
    int mirror;            // which of the two bf16 copies of S is current
    cudaEvent_t ev_before, ev_after;  // one-shot timing hook around the step kernel
    uint32_t wait_limit;   // 0: the kernels' default bound; n: waits give up after n - 1 polls (test hook)
    // projections around the core (arl2_set_projections)
    const void* w_pack;    // [d, 3 d + gate pad] bf16: W_q | W_k | W_v | W_g (zero padded)
    const void* w_o;       // [d, d] bf16
    int pack_cols;
};

namespace {

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

bool check_ctx(const arl2_ctx* ctx)
{
    if (ctx == nullptr) { set_error("context is NULL"); return false; }
    return true;
}

// the bf16 operand copy of S that is current (which = 0) or the other one (which = 1)
__nv_bfloat16* mirror_of(const arl2_ctx* ctx, int which = 0)
{
    const size_t off = ((ctx->mirror ^ which) & 1) ? ctx->lay.state_bf16_b : ctx->lay.state_bf16;
    return reinterpret_cast<__nv_bfloat16*>(ctx->ws + off);
}

// adds the launches of a helper to the context's counter; passes errors through
int account(arl2_ctx* ctx, int n)
{
    if (n < 0) return n;
    ctx->launches += (uint64_t)n;
    return ARL2_OK;
}

}  // namespace

extern "C" {

const char* arl2_version(void) { return "arl2-b200 0.1"; }

const char* arl2_last_error(void) { return g_error; }

size_t arl2_workspace_bytes(const arl2_config* cfg)
{
    if (!valid_config(cfg)) return 0;
    return make_layout(*cfg).total;
}

int arl2_create(const arl2_config* cfg, void* d_state, void* d_workspace, size_t workspace_bytes,
                void* stream, arl2_ctx** out)
{
    if (out == nullptr) { set_error("out is NULL"); return ARL2_ERR_INVALID_ARG; }
    *out = nullptr;
    if (!valid_config(cfg)) return ARL2_ERR_INVALID_ARG;
    if (d_state == nullptr || d_workspace == nullptr) {
        set_error("d_state and d_workspace must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    Layout lay = make_layout(*cfg);
    if (workspace_bytes < lay.total) {
        set_error("workspace has %zu bytes, this configuration needs %zu", workspace_bytes, lay.total);
        return ARL2_ERR_WORKSPACE;
    }
    if (reinterpret_cast<uintptr_t>(d_workspace) % kAlign != 0 ||
        reinterpret_cast<uintptr_t>(d_state) % 16 != 0) {
        set_error("d_workspace must be 256-byte aligned and d_state 16-byte aligned");
        return ARL2_ERR_WORKSPACE;
    }
    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || ndev == 0) {
        set_error("no CUDA device: %s", cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    arl2_ctx* ctx = new (std::nothrow) arl2_ctx();
    if (ctx == nullptr) { set_error("out of host memory"); return ARL2_ERR_INVALID_ARG; }
    ctx->cfg = *cfg;
    ctx->shape.B = cfg->B; ctx->shape.H = cfg->H; ctx->shape.L = cfg->L; ctx->shape.D = cfg->D;
    float scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->D);
    ctx->shape.scale_log2 = scale * 1.4426950408889634f;
    ctx->shape.eps = cfg->l2_eps > 0.0f ? cfg->l2_eps : 1e-6f;
    ctx->lay = lay;
    ctx->state = static_cast<float*>(d_state);
    ctx->ws = static_cast<uint8_t*>(d_workspace);
    ctx->wq = ctx->wk = ctx->wv = nullptr;
    ctx->rope_cos = ctx->rope_sin = nullptr;
    ctx->use_tc = tc_supported(*cfg);
    ctx->launches = 0;
    ctx->step_calls = 0;
    ctx->mirror = 0;
    ctx->w_pack = ctx->w_o = nullptr;
    ctx->pack_cols = 0;
    ctx->wait_limit = cfg->flags >> ARL2_FLAG_DEBUG_WAIT_LIMIT_SHIFT;
    ctx->ev_before = ctx->ev_after = nullptr;
    int r = account(ctx, fill_zero(ctx->ws + lay.status, kStatusWords * sizeof(uint32_t),
                                   as_stream(stream)));
    if (r == ARL2_OK && ctx->use_tc) {
        // operand copies the tensor-core kernels read: identity feature maps until
        // arl2_set_params, and the bf16 mirror of whatever the state buffer holds now
        const size_t ops[3] = {lay.wq_op, lay.wk_op, lay.wv_op};
        for (int i = 0; i < 3 && r == ARL2_OK; ++i)
            r = account(ctx, tc_prepare_map(nullptr, reinterpret_cast<__nv_bfloat16*>(ctx->ws + ops[i]),
                                            cfg->H, as_stream(stream)));
        if (r == ARL2_OK)
            r = account(ctx, state_to_bf16(ctx->state,
                                           mirror_of(ctx),
                                           (size_t)cfg->B * cfg->H * cfg->D * cfg->D, as_stream(stream)));
    }
    if (r != ARL2_OK) { delete ctx; return r; }
    *out = ctx;
    return ARL2_OK;
}

int arl2_set_params(arl2_ctx* ctx, const void* d_wphi_q, const void* d_wphi_k, const void* d_wphi_v,
                    const float* d_rope_cos, const float* d_rope_sin, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if ((d_rope_cos == nullptr) != (d_rope_sin == nullptr)) {
        set_error("rope_cos and rope_sin must both be given or both be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    if (reinterpret_cast<uintptr_t>(d_rope_cos) % 16 != 0 || reinterpret_cast<uintptr_t>(d_rope_sin) % 16 != 0) {
        set_error("rope tables must be 16-byte aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    ctx->wq = d_wphi_q; ctx->wk = d_wphi_k; ctx->wv = d_wphi_v;
    ctx->rope_cos = d_rope_cos; ctx->rope_sin = d_rope_sin;
    if (ctx->use_tc) {
        const void* src[3] = {d_wphi_q, d_wphi_k, d_wphi_v};
        const size_t ops[3] = {ctx->lay.wq_op, ctx->lay.wk_op, ctx->lay.wv_op};
        for (int i = 0; i < 3; ++i) {
            int r = account(ctx, tc_prepare_map(src[i], reinterpret_cast<__nv_bfloat16*>(ctx->ws + ops[i]),
                                                ctx->cfg.H, as_stream(stream)));
            if (r != ARL2_OK) return r;
        }
        if (d_rope_cos != nullptr) {
            int r = account(ctx, tc_prepare_rope(d_rope_cos, d_rope_sin, ctx->ws + ctx->lay.rope_h, ctx->cfg.L,
                                                 as_stream(stream)));
            if (r != ARL2_OK) return r;
        }
    }
    return ARL2_OK;
}

namespace {

bool check_step_args(const char* who, const void* d_q, const void* d_k, const void* d_v,
                     const float* d_gate_logits, const void* d_out)
{
    if (!d_q || !d_k || !d_v || !d_gate_logits || !d_out) {
        set_error("%s: q, k, v, gate_logits and out must not be NULL", who);
        return false;
    }
    if (d_out == d_q || d_out == d_k || d_out == d_v) {
        set_error("%s: out must not alias an input", who);
        return false;
    }
    if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k) |
         reinterpret_cast<uintptr_t>(d_v) | reinterpret_cast<uintptr_t>(d_out)) % 16 != 0) {
        set_error("%s: q, k, v and out must be 16-byte aligned", who);
        return false;
    }
    return true;
}

// The fused attention kernel of one pass; k_rot is K after RoPE (or K itself without a rotation).
// The buffers the step kernel needs to cut the items of its last wave into key ranges.
void attach_split(const arl2_ctx* ctx, StepArgs& a)
{
    if (!ctx->use_tc) return;
    a.split_o = reinterpret_cast<float*>(ctx->ws + ctx->lay.split_o);
    a.split_ml = reinterpret_cast<float*>(ctx->ws + ctx->lay.split_ml);
    a.split_tile_parts = kSplitTileParts;
}

int launch_step(arl2_ctx* ctx, const void* d_q, const void* k_rot, const void* d_v,
                const float* d_gate_logits, void* d_out, cudaStream_t st)
{
    StepArgs a;
    a.s = ctx->shape;
    a.q = d_q; a.k_rot = k_rot; a.v = d_v; a.gate = d_gate_logits;
    a.gate_mode = (ctx->cfg.flags & ARL2_FLAG_GATE_ELEMENTWISE) ? 2 : (ctx->cfg.flags & ARL2_FLAG_GATE_SCALAR) ? 1 : 0;
    a.state = ctx->state; a.wq = ctx->wq;
    a.rope_cos = ctx->rope_cos; a.rope_sin = ctx->rope_sin;
    a.out = d_out;
    a.wait_limit = ctx->wait_limit;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.launch_parity = (int)(ctx->step_calls & 1u);
    a.rope_h = (ctx->use_tc && ctx->rope_cos != nullptr) ? ctx->ws + ctx->lay.rope_h : nullptr;
    attach_split(ctx, a);
    cudaEvent_t e0 = ctx->ev_before, e1 = ctx->ev_after;
    ctx->ev_before = ctx->ev_after = nullptr;
    if (e0 != nullptr) cudaEventRecord(e0, st);
    int r;
    if (ctx->use_tc) {
        r = account(ctx, tc_step(a, reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wq_op),
                                 mirror_of(ctx), st));
        // the launch consumed one scheduler counter and cleared the other: only a launch that
        // really went out moves on to the other one
        if (r == ARL2_OK) ++ctx->step_calls;
    } else {
        r = account(ctx, simt_step(a, ctx->cfg.io_dtype, st));
    }
    if (e1 != nullptr) cudaEventRecord(e1, st);
    return r;
}

// K after RoPE into the workspace (one launch), or K itself when the context has no rotation.
int rotate_k(arl2_ctx* ctx, const void* d_k, const void** k_rot, cudaStream_t st)
{
    *k_rot = d_k;
    if (ctx->rope_cos == nullptr) return ARL2_OK;
    void* buf = ctx->ws + ctx->lay.k_rot;
    int r = ctx->use_tc
                ? account(ctx, tc_rope_k(ctx->shape, d_k, ctx->ws + ctx->lay.rope_h, buf, st))
                : account(ctx, simt_rope_k(ctx->shape, ctx->cfg.io_dtype, d_k, ctx->rope_cos,
                                           ctx->rope_sin, buf, st));
    if (r == ARL2_OK) *k_rot = buf;
    return r;
}

}  // namespace

int arl2_denoise_step(arl2_ctx* ctx, const void* d_q, const void* d_k, const void* d_v,
                      const float* d_gate_logits, void* d_out, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!check_step_args("denoise_step", d_q, d_k, d_v, d_gate_logits, d_out)) return ARL2_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    const void* k_rot = nullptr;
    if (int r = rotate_k(ctx, d_k, &k_rot, st)) return r;
    return launch_step(ctx, d_q, k_rot, d_v, d_gate_logits, d_out, st);
}

int arl2_denoise_step_token_level(arl2_ctx* ctx, const void* d_q, const void* d_k, const void* d_v,
                                  const float* d_gate_logits, const float* d_alpha_logits, void* d_out,
                                  void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!check_step_args("denoise_step_token_level", d_q, d_k, d_v, d_gate_logits, d_out)) return ARL2_ERR_INVALID_ARG;
    if (!ctx->use_tc || (ctx->cfg.flags & (ARL2_FLAG_GATE_SCALAR | ARL2_FLAG_GATE_ELEMENTWISE))) {
        set_error("denoise_step_token_level: built for bf16 I/O with D = 128 and the headwise gate only");
        return ARL2_ERR_UNSUPPORTED;
    }
    cudaStream_t st = as_stream(stream);
    // 1. the intra-block softmax branch alone (closed gate) ...
    const void* k_rot = nullptr;
    if (int r = rotate_k(ctx, d_k, &k_rot, st)) return r;
    if (int r = launch_step(ctx, d_q, k_rot, d_v, nullptr, d_out, st)) return r;
    // 2. ... then the causal readout adds sigmoid(g_i) Q'_i S^(i) to it
    StepArgs a;
    a.s = ctx->shape;
    a.q = d_q; a.k_rot = d_k; a.v = d_v; a.gate = d_gate_logits;
    a.state = ctx->state; a.wq = ctx->wq;
    a.rope_cos = ctx->rope_cos; a.rope_sin = ctx->rope_sin;
    a.out = d_out;
    a.wait_limit = ctx->wait_limit;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.launch_parity = 0;
    a.rope_h = ctx->rope_cos != nullptr ? ctx->ws + ctx->lay.rope_h : nullptr;
    return account(ctx, tc_token_readout(a, d_alpha_logits,
                                         reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wq_op),
                                         reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wk_op),
                                         reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wv_op), st));
}

int arl2_teacher_step(arl2_ctx* ctx, const void* d_q, const void* d_k_cache, const void* d_v_cache,
                      int32_t cache_tokens, void* d_out, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!d_q || !d_k_cache || !d_v_cache || !d_out) {
        set_error("teacher_step: q, k_cache, v_cache and out must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    if (cache_tokens < 1) {
        set_error("teacher_step: cache_tokens must be >= 1 (got %d)", cache_tokens);
        return ARL2_ERR_INVALID_ARG;
    }
    if (d_out == d_q || d_out == d_k_cache || d_out == d_v_cache) {
        set_error("teacher_step: out must not alias an input");
        return ARL2_ERR_INVALID_ARG;
    }
    if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k_cache) |
         reinterpret_cast<uintptr_t>(d_v_cache) | reinterpret_cast<uintptr_t>(d_out)) % 16 != 0) {
        set_error("teacher_step: q, k_cache, v_cache and out must be 16-byte aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    if (!ctx->use_tc) {
        set_error("teacher_step: built for bf16 I/O with D = 128 (the tensor-core context) only");
        return ARL2_ERR_UNSUPPORTED;
    }
    if ((size_t)ctx->cfg.B * cache_tokens * ctx->cfg.H * ctx->cfg.D >= ((size_t)1 << 40)) {
        set_error("teacher_step: cache too large");
        return ARL2_ERR_INVALID_ARG;
    }
    StepArgs a;
    a.s = ctx->shape;
    a.q = d_q; a.k_rot = d_k_cache; a.v = d_v_cache;
    a.gate = nullptr;                      // closed gate: the state contributes nothing
    a.state = ctx->state; a.wq = ctx->wq;
    a.rope_cos = nullptr; a.rope_sin = nullptr;
    a.out = d_out;
    a.wait_limit = ctx->wait_limit;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.launch_parity = (int)(ctx->step_calls & 1u);
    a.rope_h = nullptr;                    // the caller's Q and cache are already rotated
    a.Lk = cache_tokens;
    attach_split(ctx, a);
    cudaStream_t st = as_stream(stream);
    cudaEvent_t e0 = ctx->ev_before, e1 = ctx->ev_after;
    ctx->ev_before = ctx->ev_after = nullptr;
    if (e0 != nullptr) cudaEventRecord(e0, st);
    int r = account(ctx, tc_step(a, reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wq_op),
                                 mirror_of(ctx), st));
    if (r == ARL2_OK) ++ctx->step_calls;
    if (e1 != nullptr) cudaEventRecord(e1, st);
    return r;
}

int arl2_debug_set_wait_limit(arl2_ctx* ctx, int32_t polls)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (polls > 65534) {
        set_error("debug_set_wait_limit: polls must be <= 65534, or negative for the default (got %d)", polls);
        return ARL2_ERR_INVALID_ARG;
    }
    ctx->wait_limit = polls < 0 ? 0u : (uint32_t)polls + 1u;
    return ARL2_OK;
}

int arl2_set_profile_events(arl2_ctx* ctx, void* ev_before, void* ev_after)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    ctx->ev_before = static_cast<cudaEvent_t>(ev_before);
    ctx->ev_after = static_cast<cudaEvent_t>(ev_after);
    return ARL2_OK;
}

namespace {

// Argument block of a commit on this context (mode: 0 gated linear, 1 delta rule, 2 per-token weights).
bool fill_commit(arl2_ctx* ctx, CommitArgs& a, const void* d_k_clean, const void* d_v_clean,
                 const float* d_decay_logits, int mode, const float* d_beta, bool decay_direct)
{
    if (!d_k_clean || !d_v_clean || !d_decay_logits) {
        set_error("commit: k_clean, v_clean and decay_logits must not be NULL");
        return false;
    }
    if ((reinterpret_cast<uintptr_t>(d_k_clean) | reinterpret_cast<uintptr_t>(d_v_clean)) % 16 != 0) {
        set_error("commit: k_clean and v_clean must be 16-byte aligned");
        return false;
    }
    a.s = ctx->shape;
    a.k = d_k_clean; a.v = d_v_clean; a.decay = d_decay_logits;
    a.wk = ctx->wk; a.wv = ctx->wv;
    a.rope_cos = ctx->rope_cos; a.rope_sin = ctx->rope_sin;
    a.state = ctx->state;
    a.partials = reinterpret_cast<float*>(ctx->ws + ctx->lay.partials);
    a.partials_g = reinterpret_cast<float*>(ctx->ws + ctx->lay.partials_g);
    a.state_bf16 = ctx->use_tc ? mirror_of(ctx) : nullptr;
    a.state_bf16_next = ctx->use_tc ? mirror_of(ctx, 1) : nullptr;
    a.nsplit = ctx->lay.nsplit;
    a.nslot = ctx->lay.nslot;
    a.rope_h = (ctx->use_tc && ctx->rope_cos != nullptr) ? ctx->ws + ctx->lay.rope_h : nullptr;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.mode = mode;
    a.wait_limit = ctx->wait_limit;
    a.beta = d_beta;
    a.decay_direct = decay_direct;
    return true;
}

// The second half of a tensor-core commit: the new state goes to S and to the mirror that was not
// current, which becomes the current one.
int finish_commit(arl2_ctx* ctx, const CommitArgs& a, cudaStream_t st)
{
    int r = account(ctx, tc_commit_finish(a, st));
    if (r == ARL2_OK) ctx->mirror ^= 1;
    return r;
}

// Shared by arl2_commit, arl2_commit_delta and arl2_commit_decay_tokens.
int commit_impl(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                const float* d_decay_logits, int mode, const float* d_beta, bool decay_direct, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    CommitArgs a;
    if (!fill_commit(ctx, a, d_k_clean, d_v_clean, d_decay_logits, mode, d_beta, decay_direct))
        return ARL2_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    if (!ctx->use_tc) return account(ctx, simt_commit(a, ctx->cfg.io_dtype, st));
    int r = account(ctx, tc_commit_partials(a, reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wk_op), st));
    if (r != ARL2_OK) return r;
    return finish_commit(ctx, a, st);
}

}  // namespace

int arl2_commit(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                const float* d_decay_logits, void* stream)
{
    return commit_impl(ctx, d_k_clean, d_v_clean, d_decay_logits, 0, nullptr, false, stream);
}

int arl2_clean_pass(arl2_ctx* ctx, const void* d_q, const void* d_k_clean, const void* d_v_clean,
                    const float* d_gate_logits, const float* d_decay_logits, void* d_out, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!check_step_args("clean_pass", d_q, d_k_clean, d_v_clean, d_gate_logits, d_out)) return ARL2_ERR_INVALID_ARG;
    CommitArgs a;
    if (!fill_commit(ctx, a, d_k_clean, d_v_clean, d_decay_logits, 0, nullptr, false)) return ARL2_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    if (!ctx->use_tc) {
        // plain-FMA contexts: the same result from the two calls in sequence
        const void* k_rot = nullptr;
        if (int r = rotate_k(ctx, d_k_clean, &k_rot, st)) return r;
        if (int r = launch_step(ctx, d_q, k_rot, d_v_clean, d_gate_logits, d_out, st)) return r;
        return account(ctx, simt_commit(a, ctx->cfg.io_dtype, st));
    }
    // 1. partial sums of the state update from the K_c, V_c tiles; the same kernel writes RoPE(K_c)
    //    for the softmax branch (K_c is read and rotated once)
    const bool rotated = ctx->rope_cos != nullptr;
    a.k_rot_out = rotated ? ctx->ws + ctx->lay.k_rot : nullptr;
    int r = account(ctx, tc_commit_partials(a, reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wk_op), st));
    if (r != ARL2_OK) return r;
    // 2. the layer's output, read against the state as it still stands (Eq. 8)
    r = launch_step(ctx, d_q, rotated ? a.k_rot_out : d_k_clean, d_v_clean, d_gate_logits, d_out, st);
    if (r != ARL2_OK) return r;
    // 3. only now the state moves on
    return finish_commit(ctx, a, st);
}

int arl2_commit_tokens(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                       const float* d_alpha_logits, const float* d_beta_logits, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!(ctx->cfg.flags & ARL2_FLAG_TOKEN_GATES)) {
        set_error("commit_tokens: the context was created without ARL2_FLAG_TOKEN_GATES "
                  "(its workspace has no room for the chunk factors)");
        return ARL2_ERR_WORKSPACE;
    }
    if (!d_k_clean || !d_v_clean) {
        set_error("commit_tokens: k_clean and v_clean must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    TokenCommitArgs a;
    a.s = ctx->shape;
    a.k = d_k_clean; a.v = d_v_clean;
    a.alpha = d_alpha_logits; a.beta = d_beta_logits;
    a.wk = ctx->wk; a.wv = ctx->wv;
    a.rope_cos = ctx->rope_cos; a.rope_sin = ctx->rope_sin;
    a.state = ctx->state;
    a.state_bf16 = ctx->use_tc ? mirror_of(ctx)
                               : nullptr;
    a.w = reinterpret_cast<float*>(ctx->ws + ctx->lay.tok_w);
    a.u1 = reinterpret_cast<float*>(ctx->ws + ctx->lay.tok_u1);
    a.kh = reinterpret_cast<float*>(ctx->ws + ctx->lay.tok_kh);
    a.gc = reinterpret_cast<float*>(ctx->ws + ctx->lay.tok_gc);
    a.nchunk = ctx->lay.nchunk;
    a.decayed = (ctx->cfg.flags & ARL2_FLAG_DELTA_DECAYED_PREDICTION) != 0;
    a.wait_limit = ctx->wait_limit;
    if ((reinterpret_cast<uintptr_t>(d_k_clean) | reinterpret_cast<uintptr_t>(d_v_clean)) % 16 != 0) {
        set_error("commit_tokens: k_clean and v_clean must be 16-byte aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    if (ctx->use_tc)
        return account(ctx, tc_commit_tokens(
                                a, reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wk_op),
                                reinterpret_cast<const __nv_bfloat16*>(ctx->ws + ctx->lay.wv_op),
                                ctx->rope_cos != nullptr ? ctx->ws + ctx->lay.rope_h : nullptr,
                                reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status), as_stream(stream)));
    return account(ctx, simt_commit_tokens(a, ctx->cfg.io_dtype, as_stream(stream)));
}

int arl2_commit_delta(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                      const float* d_decay_logits, const float* d_beta_logits, void* stream)
{
    return commit_impl(ctx, d_k_clean, d_v_clean, d_decay_logits, 1, d_beta_logits, false, stream);
}

int arl2_commit_decay_tokens(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                             const float* d_alpha_logits, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!d_alpha_logits) {
        set_error("commit_decay_tokens: alpha_logits must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    float* w = reinterpret_cast<float*>(ctx->ws + ctx->lay.dec_w);
    float* total = reinterpret_cast<float*>(ctx->ws + ctx->lay.dec_total);
    int r = account(ctx, decay_weights(ctx->shape, d_alpha_logits, w, total, as_stream(stream)));
    if (r != ARL2_OK) return r;
    return commit_impl(ctx, d_k_clean, d_v_clean, total, 2, w, true, stream);
}

namespace {
// the gate logits ride in a last, zero-padded segment so that the packed width is a multiple of 256
int gate_pad_cols(int d) { return (3 * d) % 256 == 0 ? 256 : 128; }
}  // namespace

size_t arl2_projection_workspace_bytes(const arl2_config* cfg)
{
    if (!valid_config(cfg)) return 0;
    const size_t d = (size_t)cfg->H * cfg->D;
    return align_up(d * (3 * d + gate_pad_cols((int)d)) * 2);
}

int arl2_set_projections(arl2_ctx* ctx, const void* d_wq, const void* d_wk, const void* d_wv, const void* d_wg,
                         const void* d_wo, void* d_pack, size_t pack_bytes, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (!ctx->use_tc) {
        set_error("set_projections: built for bf16 I/O with D = 128 (the tensor-core context) only");
        return ARL2_ERR_UNSUPPORTED;
    }
    if (!d_wq || !d_wk || !d_wv || !d_wg || !d_wo || !d_pack) {
        set_error("set_projections: the five weights and the packing buffer must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    const size_t d = (size_t)ctx->cfg.H * ctx->cfg.D;
    const int pad = gate_pad_cols((int)d);
    const size_t cols = 3 * d + pad;
    if (pack_bytes < d * cols * 2 || reinterpret_cast<uintptr_t>(d_pack) % 256 != 0 ||
        reinterpret_cast<uintptr_t>(d_wo) % 16 != 0) {
        set_error("set_projections: the packing buffer needs %zu bytes, 256-byte aligned; W_o 16-byte aligned", d * cols * 2);
        return ARL2_ERR_WORKSPACE;
    }
    cudaStream_t st = as_stream(stream);
    uint8_t* pack = static_cast<uint8_t*>(d_pack);
    cudaError_t e = cudaMemsetAsync(pack, 0, d * cols * 2, st);
    const void* src[3] = {d_wq, d_wk, d_wv};
    for (int i = 0; i < 3 && e == cudaSuccess; ++i)
        e = cudaMemcpy2DAsync(pack + i * d * 2, cols * 2, src[i], d * 2, d * 2, d, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(pack + 3 * d * 2, cols * 2, d_wg, (size_t)ctx->cfg.H * 2, (size_t)ctx->cfg.H * 2, d,
                              cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) { set_error("set_projections: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    ctx->w_pack = d_pack;
    ctx->w_o = d_wo;
    ctx->pack_cols = (int)cols;
    return ARL2_OK;
}

int arl2_project_in(arl2_ctx* ctx, const void* d_x, void* d_q, void* d_k, void* d_v, float* d_gate_logits,
                    void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (ctx->w_pack == nullptr) { set_error("project_in: call arl2_set_projections first"); return ARL2_ERR_INVALID_ARG; }
    if (!d_x || !d_q || !d_k || !d_v || !d_gate_logits) {
        set_error("project_in: x, q, k, v and gate_logits must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    if ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k) |
         reinterpret_cast<uintptr_t>(d_v)) % 32 != 0) {
        set_error("project_in: x, q, k and v must be 32-byte aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    const int d = ctx->cfg.H * ctx->cfg.D;
    GemmArgs a;
    a.a = d_x; a.b = ctx->w_pack;
    a.M = ctx->cfg.B * ctx->cfg.L; a.N = ctx->pack_cols; a.K = d;
    a.out[0] = d_q; a.out[1] = d_k; a.out[2] = d_v;
    a.seg_cols = d; a.ld_out = d; a.n_bf16_seg = 3;
    a.out_f32 = d_gate_logits; a.f32_cols = ctx->cfg.H; a.ld_f32 = ctx->cfg.H;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.wait_limit = ctx->wait_limit;
    return account(ctx, tc_gemm(a, as_stream(stream)));
}

int arl2_project_out(arl2_ctx* ctx, const void* d_o, void* d_y, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (ctx->w_o == nullptr) { set_error("project_out: call arl2_set_projections first"); return ARL2_ERR_INVALID_ARG; }
    if (!d_o || !d_y || d_o == d_y) { set_error("project_out: o and y must be two non-NULL buffers"); return ARL2_ERR_INVALID_ARG; }
    if ((reinterpret_cast<uintptr_t>(d_o) | reinterpret_cast<uintptr_t>(d_y)) % 32 != 0) {
        set_error("project_out: o and y must be 32-byte aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    const int d = ctx->cfg.H * ctx->cfg.D;
    GemmArgs a;
    a.a = d_o; a.b = ctx->w_o;
    a.M = ctx->cfg.B * ctx->cfg.L; a.N = d; a.K = d;
    a.out[0] = d_y;
    a.seg_cols = d; a.ld_out = d; a.n_bf16_seg = 1;
    a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lay.status);
    a.wait_limit = ctx->wait_limit;
    return account(ctx, tc_gemm(a, as_stream(stream)));
}

int arl2_reset(arl2_ctx* ctx, int32_t stream_index, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (stream_index < -1 || stream_index >= ctx->cfg.B) {
        set_error("reset: stream_index %d out of range [-1, %d)", stream_index, ctx->cfg.B);
        return ARL2_ERR_INVALID_ARG;
    }
    size_t per = (size_t)ctx->cfg.H * ctx->cfg.D * ctx->cfg.D;
    size_t first = stream_index < 0 ? 0 : (size_t)stream_index * per;
    size_t count = stream_index < 0 ? per * ctx->cfg.B : per;
    cudaStream_t st = as_stream(stream);
    int r = account(ctx, fill_zero(ctx->state + first, count * sizeof(float), st));
    if (r != ARL2_OK) return r;
    if (ctx->use_tc) {
        auto* sb = mirror_of(ctx);
        r = account(ctx, fill_zero(sb + first, count * 2, st));
    }
    return r;
}

int arl2_get_state(arl2_ctx* ctx, float* dst, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (dst == nullptr) { set_error("get_state: dst is NULL"); return ARL2_ERR_INVALID_ARG; }
    size_t bytes = (size_t)ctx->cfg.B * ctx->cfg.H * ctx->cfg.D * ctx->cfg.D * sizeof(float);
    cudaError_t e = cudaMemcpyAsync(dst, ctx->state, bytes, cudaMemcpyDefault, as_stream(stream));
    if (e != cudaSuccess) {
        set_error("get_state: %s", cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    return ARL2_OK;
}

int arl2_set_state(arl2_ctx* ctx, const float* src, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    if (src == nullptr) { set_error("set_state: src is NULL"); return ARL2_ERR_INVALID_ARG; }
    size_t n = (size_t)ctx->cfg.B * ctx->cfg.H * ctx->cfg.D * ctx->cfg.D;
    cudaStream_t st = as_stream(stream);
    cudaError_t e = cudaMemcpyAsync(ctx->state, src, n * sizeof(float), cudaMemcpyDefault, st);
    if (e != cudaSuccess) {
        set_error("set_state: %s", cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    if (ctx->use_tc)
        return account(ctx, state_to_bf16(ctx->state,
                                          mirror_of(ctx),
                                          n, st));
    return ARL2_OK;
}

int arl2_sync_status(arl2_ctx* ctx, void* stream)
{
    if (!check_ctx(ctx)) return ARL2_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    uint32_t words[2] = {0, 0};
    cudaError_t e = cudaMemcpyAsync(words, ctx->ws + ctx->lay.status, sizeof(words),
                                    cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        set_error("sync_status: %s", cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    if (words[0] != 0) {
        set_error("a bounded wait inside a kernel expired (code %u, site %u)", words[0], words[1]);
        int r = account(ctx, fill_zero(ctx->ws + ctx->lay.status, kStatusWords * sizeof(uint32_t), st));
        if (r != ARL2_OK) return r;
        return ARL2_ERR_TIMEOUT;
    }
    return ARL2_OK;
}

uint64_t arl2_launch_count(const arl2_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* arl2_step_kernel_name(const arl2_ctx* ctx)
{
    if (ctx == nullptr) return "";
    return ctx->use_tc ? "tcgen05" : "simt";
}

void arl2_destroy(arl2_ctx* ctx) { delete ctx; }

}  // extern "C"
