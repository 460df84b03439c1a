// C ABI of the library (see include/mkv.h): context, workspace layout, argument checks and
// kernel dispatch.  No exception or abort crosses this file's extern "C" functions.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <initializer_list>
#include <new>

#include "../../include/mkv.h"
#include "mkv_kernels.h"

using namespace mkv;

namespace {

struct Layout {
    size_t K, V, pos, ring_q, ring_c, s_new, F, Fc, prof, part_ml, part_o, ticket, evicted, state, rows, row_shift, stage_q, stage_k, stage_v,
        stage_o, total;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Shape {
    int layers;             // layers served by this context's own arena
    int upl;                // units per layer = batch * n_kv_heads
    int B, Hkv;             // batch rows and KV heads (upl = B * Hkv)
    int U, G, D, R, C, cap, splits, T, tc_grid_size, tc_grid_layer;
    int Gq;                 // the model's GQA ratio; G is it rounded up to a power of two on the tensor-core path
    int nc;                 // ring chunks of the tensor-core kernel (1 unless the window has more than 256 rows)
    int stored;             // 1: the window tokens' attention profiles are kept as a table (profile_mode STORED)
    size_t es;
};

Layout make_layout(const Shape &s)
{
    Layout L;
    size_t o = 0;
    const size_t U = s.U, cap = s.cap, D = s.D, G = s.G, R = s.R, sp = s.splits;
    auto take = [&](size_t bytes) { const size_t at = o; o = align256(o + bytes); return at; };
    L.K = take(U * cap * D * s.es);
    L.V = take(U * cap * D * s.es);
    L.pos = take(U * cap * 4);
    L.ring_q = take(U * R * G * D * s.es);
    L.ring_c = take(U * R * G * 4);
    L.s_new = take(U * G * cap * 4);
    L.F = take(U * cap * 4);
    L.Fc = take(s.nc > 1 && !s.stored ? U * (size_t)s.nc * cap * 4 : 0);
    L.prof = take(s.stored ? U * R * cap * 4 : 0);
    L.part_ml = take(U * sp * G * 2 * 4);
    L.part_o = take(U * sp * G * D * 4);
    L.ticket = take(U * 4);
    L.evicted = take(U * 4);
    L.state = take(sizeof(DevState) * (1 + (size_t)s.layers));     // whole-stack state, then one per layer
    L.rows = take((1 + (size_t)s.layers) * 2 * s.B * 4);           // per state: the batch rows' fills, by step parity
    L.row_shift = take((size_t)s.B * 4);
    L.stage_q = take(U * (size_t)s.Gq * D * s.es);
    L.stage_k = take(U * D * s.es);
    L.stage_v = take(U * D * s.es);
    L.stage_o = take(U * (size_t)s.Gq * D * s.es);
    L.total = o;
    return L;
}

bool params_valid(const mkv_params *p)
{
    if (!p) return false;
    if (p->layers < 1 || p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1) return false;
    if (p->n_q_heads % p->n_kv_heads != 0 || p->n_q_heads / p->n_kv_heads > kMaxGroup) return false;
    if (p->head_dim != 64 && p->head_dim != 128) return false;
    if (p->C < 1 || p->R < 1) return false;
    if (p->fusion != MKV_FUSION_SUM && p->fusion != MKV_FUSION_MAX) return false;
    if (p->dtype != MKV_DTYPE_BF16 && p->dtype != MKV_DTYPE_F32) return false;
    if (p->evict_interval < 0 || p->splits < 0) return false;
    if (p->kernel != MKV_KERNEL_AUTO && p->kernel != MKV_KERNEL_SIMT && p->kernel != MKV_KERNEL_TC) return false;
    if (p->norm_mode != MKV_NORM_FROZEN && p->norm_mode != MKV_NORM_CURRENT) return false;
    if (p->profile_mode != MKV_PROFILE_RECOMPUTE && p->profile_mode != MKV_PROFILE_STORED) return false;
    if (p->full_layers < 0 || p->full_layers >= p->layers) return false;
    if (p->full_layers > 0 && p->max_tokens <= p->R) return false;
    const long long units = (long long)p->layers * p->batch * p->n_kv_heads;
    if (units > (1 << 24)) return false;
    if ((long long)p->C + p->R + (p->evict_interval > 1 ? p->evict_interval : 0) > (1 << 24)) return false;
    return true;
}

enum KernelKind { kKindSimt = 0, kKindTc = 1 };

// kernel choice and split count implied by the parameters; returns false if unsupported
bool resolve(const mkv_params *p, Shape *s, KernelKind *kind)
{
    s->layers = p->layers - p->full_layers;
    s->upl = p->batch * p->n_kv_heads;
    s->B = p->batch;
    s->Hkv = p->n_kv_heads;
    s->U = s->layers * s->upl;
    s->G = s->Gq = p->n_q_heads / p->n_kv_heads;
    s->D = p->head_dim;
    s->R = p->R;
    s->C = p->C;
    s->T = p->evict_interval > 1 ? p->evict_interval : 1;
    // with T > 1 the step that runs the policy appends first and evicts afterwards: one more slot
    s->cap = p->C + p->R + (s->T > 1 ? s->T : 0);
    s->es = p->dtype == MKV_DTYPE_F32 ? 4 : 2;
    s->nc = 1;
    s->stored = p->profile_mode == MKV_PROFILE_STORED ? 1 : 0;
    if (s->stored && (s->T > 1 || p->norm_mode != MKV_NORM_FROZEN || p->kernel == MKV_KERNEL_SIMT)) return false;
    if (s->T > 64) return false;
    if (p->norm_mode == MKV_NORM_CURRENT && s->T > 1) return false;     // the compaction drops several tokens at once
    // stored-profile mode: the decode kernel only ever needs the ring rows of the new query, whatever the window's size
    const int nc = s->stored ? 1 : tc_ring_chunks(s->G, s->R);
    const bool tc_ok = tc_shape_supported(p->dtype == MKV_DTYPE_F32, s->D, s->G, s->stored ? 1 : s->R) &&
                       (long long)s->U * nc * ((s->cap + 127) / 128) <= (1ll << 30);     // tile indices stay 32-bit
    if (p->kernel == MKV_KERNEL_TC && !tc_ok) return false;
    if (tc_ok && p->kernel != MKV_KERNEL_SIMT) {
        *kind = kKindTc;
        s->G = tc_padded_group(s->Gq);
        s->nc = nc;       // a unit appears in the schedule once per ring chunk
        // the persistent grid (148 SMs on B200; correctness does not depend on the count)
        s->tc_grid_size = tc_grid(s->U * nc, s->cap, p->splits, 148);
        // a per-layer call sees only a layer's units: ranges of about an eighth of a unit's tiles, so that a layer
        // of few units still spreads over the SMs while a unit stays within eight CTAs
        s->tc_grid_layer = tc_grid(s->upl * nc, s->cap, p->splits > 0 ? p->splits : 8, 148);
        // on a step without a policy decision only the main chunks are walked: take the worse of both schedules
        const int sp_all = std::max(tc_partials_per_unit(s->U * nc, s->cap, s->tc_grid_size),
                                    tc_partials_per_unit(s->U, s->cap, s->tc_grid_size));
        const int sp_layer = std::max(tc_partials_per_unit(s->upl * nc, s->cap, s->tc_grid_layer),
                                      tc_partials_per_unit(s->upl, s->cap, s->tc_grid_layer));
        s->splits = sp_all > sp_layer ? sp_all : sp_layer;
        return true;
    }
    if (s->stored) return false;        // the profile table is kept by the tensor-core kernel's epilogue only
    *kind = kKindSimt;
    const int max_splits = (s->cap + 31) / 32;
    int sp = p->splits > 0 ? p->splits : simt_default_splits(s->U, s->cap);
    if (sp > max_splits) sp = max_splits;
    s->splits = sp;
    s->tc_grid_size = 0;
    s->tc_grid_layer = 0;
    return true;
}

}  // namespace

struct mkv_ctx {
    mkv_params p;     // as given; p.layers counts every layer, s.layers those in this context's own arena
    Shape s;
    Layout L;
    KernelKind kind;
    TcPlan *plan, *plan_layer;
    mkv_ctx *full;    // layer-aware variant: the context of the first p.full_layers layers, which keep every token
    char *base;
    int device;       // the CUDA device the context was created on
    bool owns_workspace;
    bool prefilled;
    bool ragged;      // the batch rows' prompts had different lengths: per-row fills and position offsets are in use
    int *row_n;       // [B] host mirror of the rows' fills (ragged only)
    int *row_shift;   // [B] positions a row is behind the longest one
    long long t;      // host mirror of the device step state
    int n;
    int steps;
    int next_layer;   // per-layer calls: the layer (of this context's own) expected next; 0 at a step boundary
    int cursor;       // per-layer calls: the layer of the whole model expected next (kept by the outer context)
    int state_ahead;  // 0: whole-stack and per-layer device states level, 1: whole-stack ahead, 2: per-layer ahead
    unsigned long long launches;
    PrefillScratch prefill_scratch;
    char err[256];
};

namespace {

const char *off(const void *p, size_t bytes) { return (const char *)p + bytes; }

mkv_status fail(mkv_ctx *ctx, mkv_status st, const char *fmt, const char *detail = "")
{
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), fmt, detail);
    return st;
}

DecodeArgs make_args(const mkv_ctx *c, const void *q, const void *k, const void *v, void *out)
{
    DecodeArgs a;
    char *b = c->base;
    a.K = b + c->L.K; a.V = b + c->L.V; a.pos = (int *)(b + c->L.pos);
    a.ring_q = b + c->L.ring_q; a.ring_c = (float *)(b + c->L.ring_c);
    a.q = q; a.k_new = k; a.v_new = v; a.out = out;
    a.s_new = (float *)(b + c->L.s_new); a.F = (float *)(b + c->L.F);
    a.Fc = c->s.nc > 1 && !c->s.stored ? (float *)(b + c->L.Fc) : nullptr; a.nc = c->s.nc;
    a.prof = c->s.stored ? (float *)(b + c->L.prof) : nullptr;
    a.part_ml = (float *)(b + c->L.part_ml); a.part_o = (float *)(b + c->L.part_o);
    a.ticket = (int *)(b + c->L.ticket); a.evicted_pos = (int *)(b + c->L.evicted);
    a.st = (DevState *)(b + c->L.state);
    a.u0 = 0;
    a.U = c->s.U; a.G = c->s.G; a.Gq = c->s.Gq; a.R = c->s.R; a.C = c->s.C; a.cap = c->s.cap; a.splits = c->s.splits;
    a.fusion = c->p.fusion == MKV_FUSION_SUM ? kFusionSum : kFusionMax;
    a.T = c->s.T;
    a.norm_current = c->p.norm_mode == MKV_NORM_CURRENT ? 1 : 0;
    a.scale2 = (float)(1.4426950408889634 / sqrt((double)c->s.D));
    a.row_n = c->ragged ? (int *)(b + c->L.rows) : nullptr;
    a.row_shift = c->ragged ? (const int *)(b + c->L.row_shift) : nullptr;
    a.B = c->s.B; a.Hkv = c->s.Hkv;
    a.n_hint = c->prefilled ? c->n : 0;
    return a;
}

// Free slots and empty ring rows are read by the kernels as whole tiles (their results are
// masked afterwards), so they must hold finite numbers: zero K, V and the query ring.
bool clear_arena(mkv_ctx *c, cudaStream_t stream)
{
    const size_t kv = (size_t)c->s.U * c->s.cap * c->s.D * c->s.es, rq = (size_t)c->s.U * c->s.R * c->s.G * c->s.D * c->s.es;
    if (c->s.stored &&
        cudaMemsetAsync(c->base + c->L.prof, 0, (size_t)c->s.U * c->s.R * c->s.cap * 4, stream) != cudaSuccess) return false;
    return cudaMemsetAsync(c->base + c->L.K, 0, kv, stream) == cudaSuccess &&
           cudaMemsetAsync(c->base + c->L.V, 0, kv, stream) == cudaSuccess &&
           cudaMemsetAsync(c->base + c->L.ring_q, 0, rq, stream) == cudaSuccess;
}

// Arguments of a launch that covers one layer of the context's own: every arena pointer is moved to the layer's
// first unit, the inputs and `out` are that layer's tensors, and the layer's own step state is used.
// `row` >= 0 narrows the launch further, to that batch row's units of the layer (prompt phase of a ragged batch).
DecodeArgs make_args_layer(const mkv_ctx *c, int layer, const void *q, const void *k, const void *v, void *out, int row = -1)
{
    DecodeArgs a = make_args(c, q, k, v, out);
    const Shape &s = c->s;
    const size_t u0 = (size_t)layer * s.upl + (row >= 0 ? (size_t)row * s.Hkv : 0);
    a.K = (char *)a.K + u0 * s.cap * s.D * s.es; a.V = (char *)a.V + u0 * s.cap * s.D * s.es;
    a.pos += u0 * s.cap;
    a.ring_q = (char *)a.ring_q + u0 * s.R * s.G * s.D * s.es; a.ring_c += u0 * s.R * s.G;
    a.s_new += u0 * s.G * s.cap; a.F += u0 * s.cap;
    if (a.Fc) a.Fc += u0 * s.nc * s.cap;
    if (a.prof) a.prof += u0 * s.R * s.cap;
    a.part_ml += u0 * s.splits * s.G * 2; a.part_o += u0 * s.splits * s.G * s.D;
    a.ticket += u0; a.evicted_pos += u0;
    a.st = a.st + 1 + layer;
    if (a.row_n) a.row_n += (size_t)(1 + layer) * 2 * s.B;
    a.u0 = (int)u0;
    a.U = row >= 0 ? s.Hkv : s.upl;
    return a;
}

// Brings the whole-stack state and the per-layer states level before a call of the other kind (only at a step
// boundary: every layer has taken the same number of steps then).
mkv_status level_states(mkv_ctx *ctx, int want, cudaStream_t stream)
{
    if (ctx->state_ahead == 0 || ctx->state_ahead == want) return MKV_OK;
    DevState *st = (DevState *)(ctx->base + ctx->L.state);
    int *rows = ctx->ragged ? (int *)(ctx->base + ctx->L.rows) : nullptr;
    const int ri = 2 * ctx->s.B;
    const cudaError_t e = ctx->state_ahead == 1
        ? launch_copy_state(st + 1, ctx->s.layers, st, stream, rows ? rows + ri : nullptr, rows, ri)
        : launch_copy_state(st, 1, st + 1, stream, rows, rows ? rows + ri : nullptr, ri);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "state copy launch failed: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    ctx->state_ahead = 0;
    return MKV_OK;
}

// One decode step of the whole stack (layer < 0) or of one layer of this context's own.
mkv_status launch_step(mkv_ctx *ctx, int layer, const void *q, const void *k, const void *v, void *out, cudaStream_t stream)
{
    const mkv_status ls = level_states(ctx, layer < 0 ? 1 : 2, stream);
    if (ls != MKV_OK) return ls;
    const DecodeArgs a = layer < 0 ? make_args(ctx, q, k, v, out) : make_args_layer(ctx, layer, q, k, v, out);
    // stored-profile mode: a policy step reads its fused scores from the table first.  Launched on every step: the
    // kernel decides by the device's step state and returns at once when no policy runs, so that a recorded
    // sequence of steps stays valid when it is replayed into another phase of the sequence.
    if (ctx->s.stored) {
        const cudaError_t ef = launch_profile_fuse(a, stream);
        if (ef != cudaSuccess) return fail(ctx, MKV_CUDA, "profile launch failed: %s", cudaGetErrorString(ef));
        ctx->launches += 1;
    }
    const cudaError_t e = ctx->kind == kKindTc ? launch_decode_tc(layer < 0 ? ctx->plan : ctx->plan_layer, a, stream)
                                               : launch_decode_simt(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, stream);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "decode launch failed: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    const bool ev = step_scores(ctx->t, ctx->n, ctx->steps, ctx->s.R, ctx->s.C, ctx->s.T);
    // coarse-grained eviction: the compaction follows the steps that ran the policy (the kernel itself checks the
    // device state and does nothing if no compaction is pending)
    // (While the stream is being captured the launch is recorded after every step, so that the recorded sequence
    // stays valid when it is replayed in another phase of the eviction period.)
    bool capturing = false;
    if (ctx->s.T > 1 && !ev) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        capturing = cudaStreamIsCapturing(stream, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive;
        cudaGetLastError();
    }
    if (ctx->s.T > 1 && (ev || capturing)) {
        const cudaError_t e2 = launch_compact(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, stream);
        if (e2 != cudaSuccess) return fail(ctx, MKV_CUDA, "compaction launch failed: %s", cudaGetErrorString(e2));
        ctx->launches += 1;
    }
    if (layer >= 0) {
        ctx->state_ahead = 2;
        ctx->next_layer = layer + 1 < ctx->s.layers ? layer + 1 : 0;
        if (ctx->next_layer != 0) return MKV_OK;          // the step is complete once its last layer has run
    } else {
        ctx->state_ahead = 1;
    }
    if (ctx->ragged) {       // every row by its own fill; the uniform fill is the largest
        int nmax = 0;
        for (int b = 0; b < ctx->s.B; ++b) {
            if (!step_scores(ctx->t - ctx->row_shift[b], ctx->row_n[b], ctx->steps, ctx->s.R, ctx->s.C, ctx->s.T)) ctx->row_n[b] += 1;
            nmax = std::max(nmax, ctx->row_n[b]);
        }
        ctx->n = nmax;
    } else if (!ev) {
        ctx->n += 1;
    } else if (ctx->s.T > 1) {
        ctx->n = ctx->s.C + ctx->s.R;
    }
    ctx->t += 1;
    ctx->steps += 1;
    return MKV_OK;
}

// ---- the calls on one context's own layers ------------------------------------------------------------------
mkv_status core_create(mkv_ctx **out, const mkv_params *p, void *workspace, size_t workspace_bytes)
{
    *out = nullptr;
    Shape s;
    KernelKind kind;
    if (!resolve(p, &s, &kind)) return MKV_UNSUPPORTED;
    const Layout L = make_layout(s);
    if (workspace && workspace_bytes < L.total) return MKV_OOM;
    mkv_ctx *c = new (std::nothrow) mkv_ctx;
    if (!c) return MKV_OOM;
    memset(c, 0, sizeof(*c));
    c->p = *p; c->s = s; c->L = L; c->kind = kind;
    c->row_n = new (std::nothrow) int[2 * (size_t)s.B];
    if (!c->row_n) { delete c; return MKV_OOM; }
    c->row_shift = c->row_n + s.B;
    if (cudaGetDevice(&c->device) != cudaSuccess) { cudaGetLastError(); delete[] c->row_n; delete c; return MKV_CUDA; }
    if (workspace) {
        c->base = (char *)workspace;
    } else {
        void *mem = nullptr;
        if (cudaMalloc(&mem, L.total) != cudaSuccess) {
            cudaGetLastError();
            delete[] c->row_n;
            delete c;
            return MKV_OOM;
        }
        c->base = (char *)mem;
        c->owns_workspace = true;
    }
    if (kind == kKindTc) {
        const DecodeArgs a = make_args(c, nullptr, nullptr, nullptr, nullptr);
        char msg[200] = "";
        cudaError_t e = tc_plan_create(&c->plan, a, s.tc_grid_size, p->wait_limit_cycles, true, msg, sizeof(msg));
        if (e == cudaSuccess) e = tc_plan_create(&c->plan_layer, a, s.tc_grid_layer, p->wait_limit_cycles, false, msg, sizeof(msg));
        if (e != cudaSuccess) {
            cudaGetLastError();
            if (c->plan) tc_plan_destroy(c->plan);
            if (c->owns_workspace) cudaFree(c->base);
            delete[] c->row_n;
            delete c;
            return e == cudaErrorMemoryAllocation ? MKV_OOM : MKV_CUDA;
        }
    }
    *out = c;
    return MKV_OK;
}

void core_destroy(mkv_ctx *ctx)
{
    if (!ctx) return;
    if (ctx->plan) tc_plan_destroy(ctx->plan);
    if (ctx->plan_layer) tc_plan_destroy(ctx->plan_layer);
    if (ctx->prefill_scratch.ptr) cudaFree(ctx->prefill_scratch.ptr);
    if (ctx->owns_workspace && ctx->base) cudaFree(ctx->base);
    delete[] ctx->row_n;
    delete ctx;
}

// use_static: scratch in the library's fixed device array instead of an allocation
mkv_status core_prefill(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, cudaStream_t stream,
                        bool use_static, const char *who)
{
    char where[64];
    snprintf(where, sizeof(where), "%s", who);
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "%s: context already holds a sequence", where);
    const int Rw = prompt_len < ctx->s.R ? prompt_len : ctx->s.R;
    if (use_static) {
        const size_t need = ((size_t)Rw * ctx->s.G + 1) * (size_t)prompt_len;
        if (need > prefill_static_max_floats()) {
            snprintf(ctx->err, sizeof(ctx->err),
                     "mkv_prefill_static: one unit needs (min(R,P)*G + 1) * prompt_len = %zu floats of scratch, the fixed "
                     "array holds %zu; use mkv_prefill for this prompt", need, prefill_static_max_floats());
            return MKV_UNSUPPORTED;
        }
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev != ctx->device)
            return fail(ctx, MKV_INVALID_ARG, "%s: the current CUDA device is not the one the context was created on", where);
    }
    ctx->ragged = false;
    const DecodeArgs a = make_args(ctx, nullptr, nullptr, nullptr, nullptr);
    if (!clear_arena(ctx, stream)) return fail(ctx, MKV_CUDA, "%s: clearing the arena failed", where);
    const bool f32 = ctx->p.dtype == MKV_DTYPE_F32;
    const int n_states = 1 + ctx->s.layers;
    const cudaError_t e = use_static
        ? run_prefill_static(a, f32, ctx->s.D, k, v, q_window, prompt_len, stream, &ctx->launches, ctx->device, n_states)
        : run_prefill(a, f32, ctx->s.D, k, v, q_window, prompt_len, stream, &ctx->launches, &ctx->prefill_scratch, n_states);
    if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return fail(ctx, MKV_OOM, "%s: no memory for scratch", where); }
    if (e == cudaErrorLaunchTimeout) { cudaGetLastError(); return fail(ctx, MKV_DEVICE_TIMEOUT, "%s: a device-side wait of the prompt phase ran out", where); }
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "prompt phase: %s", cudaGetErrorString(e));
    ctx->n = (prompt_len - Rw > ctx->s.C) ? ctx->s.C + Rw : prompt_len;
    if (ctx->s.stored) {        // the window rows' profiles over the kept tokens
        cudaError_t ep = launch_prefill_profile(a, ctx->n, prompt_len, stream);
        if (ep == cudaSuccess) ep = cudaStreamSynchronize(stream);
        if (ep != cudaSuccess) return fail(ctx, MKV_CUDA, "prompt phase (profile table): %s", cudaGetErrorString(ep));
        ctx->launches += 1;
    }
    ctx->t = prompt_len;
    ctx->steps = 0;
    ctx->next_layer = 0;
    ctx->state_ahead = 0;
    ctx->prefilled = true;
    return MKV_OK;
}

// Prompt phase of a batch whose rows have prompts of different lengths (tensors padded to `padded_len` tokens): every
// row goes through the prompt phase by itself, layer by layer, then the common step state is set.
mkv_status core_prefill_ragged(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, const int32_t *prompt_len,
                               int padded_len, cudaStream_t stream)
{
    const Shape &s = ctx->s;
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_prefill_ragged: context already holds a sequence%s");
    if (s.T > 1) return fail(ctx, MKV_UNSUPPORTED, "mkv_prefill_ragged: not available with coarse-grained eviction%s");
    if (s.stored) return fail(ctx, MKV_UNSUPPORTED, "mkv_prefill_ragged: not available with the stored attention profile%s");
    if (s.nc > 1) return fail(ctx, MKV_UNSUPPORTED, "mkv_prefill_ragged: not available with a window of more than 256 ring rows on the tensor-core kernel; create the context with the CUDA-core kernel%s");
    int longest = 0;
    for (int b = 0; b < s.B; ++b) longest = std::max(longest, (int)prompt_len[b]);
    ctx->ragged = true;          // make_args hands the row arrays to the kernels from here on
    if (!clear_arena(ctx, stream)) return fail(ctx, MKV_CUDA, "mkv_prefill_ragged: clearing the arena failed%s");
    const bool f32 = ctx->p.dtype == MKV_DTYPE_F32;
    const int qw_stride = padded_len < s.R ? padded_len : s.R;
    int nmax = 0;
    for (int b = 0; b < s.B; ++b) {
        const int P = prompt_len[b], Rw = P < s.R ? P : s.R;
        ctx->row_n[b] = (P - Rw > s.C) ? s.C + Rw : P;
        ctx->row_shift[b] = longest - P;
        nmax = std::max(nmax, ctx->row_n[b]);
    }
    for (int layer = 0; layer < s.layers; ++layer) {
        for (int b = 0; b < s.B; ++b) {
            const DecodeArgs a = make_args_layer(ctx, layer, nullptr, nullptr, nullptr, nullptr, b);
            const size_t unit = ((size_t)layer * s.B + b) * s.Hkv;
            const PrefillRow row = {padded_len, qw_stride, ctx->row_shift[b]};
            const cudaError_t e = run_prefill(a, f32, s.D, off(k, unit * padded_len * s.D * s.es), off(v, unit * padded_len * s.D * s.es),
                                              off(q_window, unit * s.Gq * qw_stride * s.D * s.es), prompt_len[b], stream,
                                              &ctx->launches, &ctx->prefill_scratch, 0, &row);
            if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return fail(ctx, MKV_OOM, "mkv_prefill_ragged: no memory for scratch%s"); }
            if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "prompt phase: %s", cudaGetErrorString(e));
        }
    }
    // the rows' fills for every state and both step parities, their offsets, then the common state
    const int ns = 1 + s.layers;
    int *rows_h = new (std::nothrow) int[(size_t)ns * 2 * s.B];
    if (!rows_h) return fail(ctx, MKV_OOM, "mkv_prefill_ragged: out of host memory%s");
    for (int i = 0; i < ns * 2; ++i) memcpy(rows_h + (size_t)i * s.B, ctx->row_n, sizeof(int) * s.B);
    cudaError_t e = cudaMemcpyAsync(ctx->base + ctx->L.rows, rows_h, sizeof(int) * ns * 2 * s.B, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->base + ctx->L.row_shift, ctx->row_shift, sizeof(int) * s.B, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = launch_set_state((DevState *)(ctx->base + ctx->L.state), ns, (long long)longest, nmax, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    delete[] rows_h;
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "prompt phase: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    ctx->n = nmax;
    ctx->t = longest;
    ctx->steps = 0;
    ctx->next_layer = 0;
    ctx->state_ahead = 0;
    ctx->prefilled = true;
    return MKV_OK;
}

mkv_status core_sync(mkv_ctx *ctx, cudaStream_t stream)
{
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_sync: %s", cudaGetErrorString(e));
    // whole-stack state first, then the per-layer states
    const int ns = 1 + ctx->s.layers;
    DevState *st = new (std::nothrow) DevState[ns];
    if (!st) return fail(ctx, MKV_OOM, "mkv_sync: out of host memory%s");
    e = cudaMemcpy(st, ctx->base + ctx->L.state, sizeof(DevState) * ns, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { delete[] st; return fail(ctx, MKV_CUDA, "mkv_sync: %s", cudaGetErrorString(e)); }
    int err = kErrNone;
    for (int i = 0; i < ns && err == kErrNone; ++i) err = st[i].err;
    const DevState cur = st[ctx->state_ahead == 2 ? 1 : 0];
    delete[] st;
    if (err == kErrCacheOverflow)
        return fail(ctx, MKV_BAD_STATE, "a decode step found no free slot: coarse-grained eviction ran out of step%s");
    if (err != kErrNone) {
        char code[32];
        snprintf(code, sizeof(code), " (wait code %d)", err);
        return fail(ctx, MKV_DEVICE_TIMEOUT, "a device-side wait ran out of iterations%s", code);
    }
    // the device-resident state is authoritative (steps replayed from a CUDA graph advance
    // it without passing through this library); the host mirror follows it at a step boundary
    if (ctx->prefilled && ctx->next_layer == 0) {
        ctx->t = cur.t; ctx->n = cur.n; ctx->steps = cur.steps;
        if (ctx->ragged) {       // the rows' fills of that state, in the buffer of the current step parity
            const size_t at = ((size_t)(ctx->state_ahead == 2 ? 1 : 0) * 2 + (cur.steps & 1)) * ctx->s.B;
            e = cudaMemcpy(ctx->row_n, (const int *)(ctx->base + ctx->L.rows) + at, sizeof(int) * ctx->s.B, cudaMemcpyDeviceToHost);
            if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_sync: %s", cudaGetErrorString(e));
        }
    }
    return MKV_OK;
}

// fill and next position of batch row `row` as layer `layer` of this context sees them now
void core_row_state(const mkv_ctx *ctx, int layer, int row, int32_t *count, int64_t *next_pos)
{
    const Shape &s = ctx->s;
    const bool ahead = layer < ctx->next_layer;     // the layer has taken the step that is under way
    const int sh = ctx->ragged ? ctx->row_shift[row] : 0;
    const int n = ctx->ragged ? ctx->row_n[row] : ctx->n;
    const bool ev = step_scores(ctx->t - sh, n, ctx->steps, s.R, s.C, s.T);
    if (count) *count = !ahead ? n : (!ev ? n + 1 : (s.T > 1 ? s.C + s.R : n));
    if (next_pos) *next_pos = ctx->t - sh + (ahead ? 1 : 0);
}

void core_view(mkv_ctx *ctx, int layer, mkv_view *view)
{
    const size_t u0 = (size_t)ctx->s.upl * layer;
    const Shape &s = ctx->s;
    char *b = ctx->base;
    view->K = b + ctx->L.K + u0 * s.cap * s.D * s.es;
    view->V = b + ctx->L.V + u0 * s.cap * s.D * s.es;
    view->pos = (int32_t *)(b + ctx->L.pos) + u0 * s.cap;
    view->F = (float *)(b + ctx->L.F) + u0 * s.cap;
    view->evicted_pos = (int32_t *)(b + ctx->L.evicted) + u0;
    view->ring_q = b + ctx->L.ring_q + u0 * s.R * s.G * s.D * s.es;
    view->ring_c = (float *)(b + ctx->L.ring_c) + u0 * s.R * s.G;
    // between the per-layer calls of a step the layers below next_layer have taken the step already
    const bool ahead = layer < ctx->next_layer;
    const bool ev = step_scores(ctx->t, ctx->n, ctx->steps, s.R, s.C, s.T);
    view->count = !ahead ? ctx->n : (!ev ? ctx->n + 1 : (s.T > 1 ? s.C + s.R : ctx->n));
    if (ctx->ragged) {      // the largest fill among the rows; mkv_row_state gives each row's own
        int32_t cnt[1];
        view->count = 0;
        for (int r = 0; r < s.B; ++r) { core_row_state(ctx, layer, r, cnt, nullptr); view->count = std::max(view->count, cnt[0]); }
    }
    view->capacity = s.cap;
    view->group_stride = s.G;
    view->next_pos = ctx->t + (ahead ? 1 : 0);
}

// byte offsets of the first own layer inside whole-model tensors
size_t q_bytes_per_layer(const mkv_ctx *c) { return (size_t)c->p.batch * c->p.n_q_heads * c->s.D * c->s.es; }
size_t kv_bytes_per_layer(const mkv_ctx *c) { return (size_t)c->p.batch * c->p.n_kv_heads * c->s.D * c->s.es; }

}  // namespace

extern "C" {

void mkv_default_params(mkv_params *p)
{
    if (!p) return;
    memset(p, 0, sizeof(*p));
    p->fusion = MKV_FUSION_SUM;
    p->dtype = MKV_DTYPE_BF16;
    p->evict_interval = 1;
    p->kernel = MKV_KERNEL_AUTO;
}

// the parameters of the context that serves the first full_layers layers: a cache that holds max_tokens
static mkv_params full_layer_params(const mkv_params *p)
{
    mkv_params c = *p;
    c.layers = p->full_layers;
    c.full_layers = 0;
    c.max_tokens = 0;
    c.C = p->max_tokens - p->R;
    c.evict_interval = 1;
    c.profile_mode = MKV_PROFILE_RECOMPUTE;      // those layers keep everything: there is no score to take
    c.workspace = nullptr;
    c.workspace_bytes = 0;
    return c;
}

size_t mkv_workspace_bytes(const mkv_params *p)
{
    if (!params_valid(p)) return 0;
    Shape s;
    KernelKind kind;
    if (!resolve(p, &s, &kind)) return 0;
    size_t total = align256(make_layout(s).total);
    if (p->full_layers > 0) {
        const mkv_params c = full_layer_params(p);
        if (!params_valid(&c) || !resolve(&c, &s, &kind)) return 0;
        total += align256(make_layout(s).total);
    }
    return total;
}

mkv_status mkv_create_ex(mkv_ctx **out, const mkv_params *p)
{
    if (!out) return MKV_INVALID_ARG;
    *out = nullptr;
    if (!params_valid(p)) return MKV_INVALID_ARG;
    if (p->workspace && ((uintptr_t)p->workspace & 255) != 0) return MKV_INVALID_ARG;
    const size_t need = mkv_workspace_bytes(p);
    if (need == 0) return MKV_UNSUPPORTED;
    if (p->workspace && p->workspace_bytes < need) return MKV_OOM;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        cudaGetLastError();
        return MKV_CUDA;
    }
    Shape s;
    KernelKind kind;
    resolve(p, &s, &kind);
    const size_t own_bytes = align256(make_layout(s).total);
    mkv_ctx *c = nullptr;
    mkv_status st = core_create(&c, p, p->workspace, p->workspace ? own_bytes : 0);
    if (st != MKV_OK) return st;
    if (p->full_layers > 0) {
        const mkv_params cp = full_layer_params(p);
        st = core_create(&c->full, &cp, p->workspace ? (char *)p->workspace + own_bytes : nullptr,
                         p->workspace ? need - own_bytes : 0);
        if (st != MKV_OK) { core_destroy(c); return st; }
    }
    *out = c;
    return MKV_OK;
}

mkv_status mkv_create(mkv_ctx **out, int layers, int batch, int n_q_heads, int n_kv_heads, int head_dim, int C, int R,
                      mkv_fusion fusion)
{
    mkv_params p;
    mkv_default_params(&p);
    p.layers = layers; p.batch = batch; p.n_q_heads = n_q_heads; p.n_kv_heads = n_kv_heads;
    p.head_dim = head_dim; p.C = C; p.R = R; p.fusion = fusion;
    return mkv_create_ex(out, &p);
}

void mkv_destroy(mkv_ctx *ctx)
{
    if (!ctx) return;
    core_destroy(ctx->full);
    core_destroy(ctx);
}

static mkv_status prefill_any(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, void *stream,
                              bool use_static, const char *who)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!k || !v || !q_window) return fail(ctx, MKV_INVALID_ARG, "%s: NULL tensor", who);
    if (prompt_len < 1 || prompt_len > (1 << 24)) return fail(ctx, MKV_INVALID_ARG, "%s: prompt_len out of range", who);
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "%s: context already holds a sequence", who);
    const int Rw = prompt_len < ctx->s.R ? prompt_len : ctx->s.R;
    size_t off_kv = 0, off_q = 0;
    if (ctx->full) {
        if (prompt_len > ctx->p.max_tokens) return fail(ctx, MKV_INVALID_ARG, "%s: the prompt is longer than max_tokens", who);
        const mkv_status st = core_prefill(ctx->full, k, v, q_window, prompt_len, (cudaStream_t)stream, use_static, who);
        if (st != MKV_OK) { snprintf(ctx->err, sizeof(ctx->err), "%s", ctx->full->err); return st; }
        off_kv = kv_bytes_per_layer(ctx) * prompt_len * ctx->p.full_layers;
        off_q = q_bytes_per_layer(ctx) * Rw * ctx->p.full_layers;
    }
    return core_prefill(ctx, off(k, off_kv), off(v, off_kv), off(q_window, off_q), prompt_len, (cudaStream_t)stream, use_static, who);
}

mkv_status mkv_reset(mkv_ctx *ctx)
{
    if (!ctx) return MKV_INVALID_ARG;
    for (mkv_ctx *c : {ctx, ctx->full}) {
        if (!c) continue;
        c->prefilled = false;
        c->ragged = false;
        c->t = 0; c->n = 0; c->steps = 0; c->next_layer = 0; c->state_ahead = 0; c->cursor = 0;
    }
    return MKV_OK;
}

mkv_status mkv_prefill(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, void *stream)
{
    return prefill_any(ctx, k, v, q_window, prompt_len, stream, false, "mkv_prefill");
}

mkv_status mkv_prefill_static(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, void *stream)
{
    return prefill_any(ctx, k, v, q_window, prompt_len, stream, true, "mkv_prefill_static");
}

mkv_status mkv_prefill_ragged(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, const int32_t *prompt_len,
                              int padded_len, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!k || !v || !q_window || !prompt_len) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_ragged: NULL argument%s");
    if (padded_len < 1 || padded_len > (1 << 24)) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_ragged: padded_len out of range%s");
    for (int b = 0; b < ctx->p.batch; ++b)
        if (prompt_len[b] < 1 || prompt_len[b] > padded_len)
            return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_ragged: every prompt_len must lie in [1, padded_len]%s");
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_prefill_ragged: context already holds a sequence%s");
    const int qw = padded_len < ctx->s.R ? padded_len : ctx->s.R;
    size_t off_kv = 0, off_q = 0;
    if (ctx->full) {
        for (int b = 0; b < ctx->p.batch; ++b)
            if (prompt_len[b] > ctx->p.max_tokens) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_ragged: a prompt is longer than max_tokens%s");
        const mkv_status st = core_prefill_ragged(ctx->full, k, v, q_window, prompt_len, padded_len, (cudaStream_t)stream);
        if (st != MKV_OK) { snprintf(ctx->err, sizeof(ctx->err), "%s", ctx->full->err); return st; }
        off_kv = kv_bytes_per_layer(ctx) * padded_len * ctx->p.full_layers;
        off_q = q_bytes_per_layer(ctx) * qw * ctx->p.full_layers;
    }
    return core_prefill_ragged(ctx, off(k, off_kv), off(v, off_kv), off(q_window, off_q), prompt_len, padded_len, (cudaStream_t)stream);
}

mkv_status mkv_row_state(mkv_ctx *ctx, int layer, int32_t *count, int64_t *next_pos)
{
    if (!ctx || (!count && !next_pos)) return MKV_INVALID_ARG;
    if (layer < 0 || layer >= ctx->p.layers) return fail(ctx, MKV_INVALID_ARG, "mkv_row_state: layer out of range%s");
    const mkv_ctx *c = layer < ctx->p.full_layers ? ctx->full : ctx;
    const int l = layer < ctx->p.full_layers ? layer : layer - ctx->p.full_layers;
    for (int b = 0; b < ctx->p.batch; ++b) core_row_state(c, l, b, count ? count + b : nullptr, next_pos ? next_pos + b : nullptr);
    return MKV_OK;
}

mkv_status mkv_decode_step(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *out, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!q || !k_new || !v_new || !out) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_step: NULL tensor%s");
    if (!ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_decode_step: call mkv_prefill first%s");
    if (ctx->cursor != 0)
        return fail(ctx, MKV_BAD_STATE, "mkv_decode_step: a step begun with mkv_decode_step_layer has layers left%s");
    if (ctx->t >= 0x7fffffffLL) return fail(ctx, MKV_UNSUPPORTED, "mkv_decode_step: position exceeds int32%s");
    size_t oq = 0, okv = 0;
    if (ctx->full) {
        const mkv_status st = launch_step(ctx->full, -1, q, k_new, v_new, out, (cudaStream_t)stream);
        if (st != MKV_OK) { snprintf(ctx->err, sizeof(ctx->err), "%s", ctx->full->err); return st; }
        oq = q_bytes_per_layer(ctx) * ctx->p.full_layers;
        okv = kv_bytes_per_layer(ctx) * ctx->p.full_layers;
    }
    return launch_step(ctx, -1, off(q, oq), off(k_new, okv), off(v_new, okv), (char *)out + oq, (cudaStream_t)stream);
}

mkv_status mkv_decode_step_layer(mkv_ctx *ctx, int layer, const void *q, const void *k_new, const void *v_new, void *out,
                                 void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!q || !k_new || !v_new || !out) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_step_layer: NULL tensor%s");
    if (!ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_decode_step_layer: call mkv_prefill first%s");
    if (layer < 0 || layer >= ctx->p.layers) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_step_layer: layer out of range%s");
    if (ctx->t >= 0x7fffffffLL) return fail(ctx, MKV_UNSUPPORTED, "mkv_decode_step_layer: position exceeds int32%s");
    // the layers of a step come in order 0, 1, ..., layers - 1
    const int fl = ctx->p.full_layers;
    if (layer != ctx->cursor) return fail(ctx, MKV_BAD_STATE, "mkv_decode_step_layer: layers must be called in order within a step%s");
    mkv_status st;
    if (layer < fl) {
        st = launch_step(ctx->full, layer, q, k_new, v_new, out, (cudaStream_t)stream);
        if (st != MKV_OK) snprintf(ctx->err, sizeof(ctx->err), "%s", ctx->full->err);
    } else {
        st = launch_step(ctx, layer - fl, q, k_new, v_new, out, (cudaStream_t)stream);
    }
    if (st == MKV_OK) ctx->cursor = layer + 1 < ctx->p.layers ? layer + 1 : 0;
    return st;
}

mkv_status mkv_decode_steps(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *out, int n_steps,
                            void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (n_steps < 0) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_steps: negative n_steps%s");
    const size_t qb = q_bytes_per_layer(ctx) * ctx->p.layers, kb = kv_bytes_per_layer(ctx) * ctx->p.layers;
    for (int i = 0; i < n_steps; ++i) {
        const mkv_status st = mkv_decode_step(ctx, (const char *)q + i * qb, (const char *)k_new + i * kb,
                                              (const char *)v_new + i * kb, (char *)out + i * qb, stream);
        if (st != MKV_OK) return st;
    }
    return MKV_OK;
}

mkv_status mkv_decode_step_host(mkv_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host,
                                void *out_host, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!q_host || !k_new_host || !v_new_host || !out_host) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_step_host: NULL buffer%s");
    if (!ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_decode_step_host: call mkv_prefill first%s");
    if (ctx->full) return fail(ctx, MKV_UNSUPPORTED, "mkv_decode_step_host: not available with full_layers; copy the inputs and call mkv_decode_step%s");
    cudaStream_t s = (cudaStream_t)stream;
    const size_t qb = (size_t)ctx->s.U * ctx->s.Gq * ctx->s.D * ctx->s.es, kb = (size_t)ctx->s.U * ctx->s.D * ctx->s.es;
    char *b = ctx->base;
    // Pinned host buffers are reachable from the device: the tensor-core kernel then reads q, k_new, v_new and
    // writes `out` in place over the interconnect (a few hundred KB per step, read once or twice), which saves
    // four copy launches per step.  Anything else goes through the staging buffers.
    if (ctx->kind == kKindTc) {
        const void *hp[4] = {q_host, k_new_host, v_new_host, out_host};
        void *dp[4] = {nullptr, nullptr, nullptr, nullptr};
        bool mapped = true;
        for (int i = 0; i < 4 && mapped; ++i) {
            cudaPointerAttributes at;
            mapped = cudaPointerGetAttributes(&at, hp[i]) == cudaSuccess && at.type == cudaMemoryTypeHost &&
                     cudaHostGetDevicePointer(&dp[i], const_cast<void *>(hp[i]), 0) == cudaSuccess && dp[i] != nullptr;
        }
        cudaGetLastError();     // a failed query of pageable memory is not an error of this call
        if (mapped) return mkv_decode_step(ctx, dp[0], dp[1], dp[2], dp[3], stream);
    }
    cudaError_t e = cudaMemcpyAsync(b + ctx->L.stage_q, q_host, qb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b + ctx->L.stage_k, k_new_host, kb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b + ctx->L.stage_v, v_new_host, kb, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_decode_step_host: %s", cudaGetErrorString(e));
    const mkv_status st = mkv_decode_step(ctx, b + ctx->L.stage_q, b + ctx->L.stage_k, b + ctx->L.stage_v,
                                          b + ctx->L.stage_o, stream);
    if (st != MKV_OK) return st;
    e = cudaMemcpyAsync(out_host, b + ctx->L.stage_o, qb, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_decode_step_host: %s", cudaGetErrorString(e));
    return MKV_OK;
}

mkv_status mkv_cache_view(mkv_ctx *ctx, int layer, mkv_view *view)
{
    if (!ctx || !view) return MKV_INVALID_ARG;
    if (layer < 0 || layer >= ctx->p.layers) return fail(ctx, MKV_INVALID_ARG, "mkv_cache_view: layer out of range%s");
    if (layer < ctx->p.full_layers) core_view(ctx->full, layer, view);
    else core_view(ctx, layer - ctx->p.full_layers, view);
    return MKV_OK;
}

mkv_status mkv_sync(mkv_ctx *ctx, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (ctx->full) {
        const mkv_status st = core_sync(ctx->full, (cudaStream_t)stream);
        if (st != MKV_OK) { snprintf(ctx->err, sizeof(ctx->err), "%s", ctx->full->err); return st; }
    }
    return core_sync(ctx, (cudaStream_t)stream);
}

const char *mkv_last_error(const mkv_ctx *ctx) { return ctx ? ctx->err : ""; }

uint64_t mkv_launch_count(const mkv_ctx *ctx) { return ctx ? ctx->launches + (ctx->full ? ctx->full->launches : 0) : 0; }

const char *mkv_kernel_name(const mkv_ctx *ctx) { return (ctx && ctx->kind == kKindTc) ? "tc" : "simt"; }

}  // extern "C"
