// C ABI of the library (see include/mkv.h): context, workspace layout, argument checks and
// kernel dispatch.  No exception or abort crosses this file's extern "C" functions.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "../../include/mkv.h"
#include "mkv_kernels.h"

using namespace mkv;

namespace {

struct Layout {
    size_t K, V, pos, ring_q, ring_c, s_new, F, part_ml, part_o, ticket, evicted, state, stage_q, stage_k, stage_v,
        stage_o, total;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Shape {
    int U, G, D, R, C, cap, splits, T, tc_grid_size;
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
    L.part_ml = take(U * sp * G * 2 * 4);
    L.part_o = take(U * sp * G * D * 4);
    L.ticket = take(U * 4);
    L.evicted = take(U * 4);
    L.state = take(sizeof(DevState));
    L.stage_q = take(U * G * D * s.es);
    L.stage_k = take(U * D * s.es);
    L.stage_v = take(U * D * s.es);
    L.stage_o = take(U * G * D * s.es);
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
    const long long units = (long long)p->layers * p->batch * p->n_kv_heads;
    if (units > (1 << 24)) return false;
    if ((long long)p->C + p->R + (p->evict_interval > 1 ? p->evict_interval : 0) > (1 << 24)) return false;
    return true;
}

enum KernelKind { kKindSimt = 0, kKindTc = 1 };

// kernel choice and split count implied by the parameters; returns false if unsupported
bool resolve(const mkv_params *p, Shape *s, KernelKind *kind)
{
    s->U = p->layers * p->batch * p->n_kv_heads;
    s->G = p->n_q_heads / p->n_kv_heads;
    s->D = p->head_dim;
    s->R = p->R;
    s->C = p->C;
    s->T = p->evict_interval > 1 ? p->evict_interval : 1;
    // with T > 1 the step that runs the policy appends first and evicts afterwards: one more slot
    s->cap = p->C + p->R + (s->T > 1 ? s->T : 0);
    s->es = p->dtype == MKV_DTYPE_F32 ? 4 : 2;
    if (s->T > 64) return false;
    const bool tc_ok = tc_shape_supported(p->dtype == MKV_DTYPE_F32, s->D, s->G, s->R) &&
                       (long long)s->U * ((s->cap + 127) / 128) <= (1ll << 30);     // tile indices stay 32-bit
    if (p->kernel == MKV_KERNEL_TC && !tc_ok) return false;
    if (tc_ok && p->kernel != MKV_KERNEL_SIMT) {
        *kind = kKindTc;
        // the persistent grid (148 SMs on B200; correctness does not depend on the count)
        s->tc_grid_size = tc_grid(s->U, s->cap, p->splits, 148);
        s->splits = tc_partials_per_unit(s->U, s->cap, s->tc_grid_size);
        return true;
    }
    *kind = kKindSimt;
    const int max_splits = (s->cap + 31) / 32;
    int sp = p->splits > 0 ? p->splits : simt_default_splits(s->U, s->cap);
    if (sp > max_splits) sp = max_splits;
    s->splits = sp;
    s->tc_grid_size = 0;
    return true;
}

}  // namespace

struct mkv_ctx {
    mkv_params p;
    Shape s;
    Layout L;
    KernelKind kind;
    TcPlan *plan;
    char *base;
    bool owns_workspace;
    bool prefilled;
    long long t;      // host mirror of the device step state
    int n;
    int steps;
    unsigned long long launches;
    PrefillScratch prefill_scratch;
    char err[256];
};

namespace {

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
    a.part_ml = (float *)(b + c->L.part_ml); a.part_o = (float *)(b + c->L.part_o);
    a.ticket = (int *)(b + c->L.ticket); a.evicted_pos = (int *)(b + c->L.evicted);
    a.st = (DevState *)(b + c->L.state);
    a.U = c->s.U; a.G = c->s.G; a.R = c->s.R; a.C = c->s.C; a.cap = c->s.cap; a.splits = c->s.splits;
    a.fusion = c->p.fusion == MKV_FUSION_SUM ? kFusionSum : kFusionMax;
    a.T = c->s.T;
    a.scale2 = (float)(1.4426950408889634 / sqrt((double)c->s.D));
    return a;
}

// Free slots and empty ring rows are read by the kernels as whole tiles (their results are
// masked afterwards), so they must hold finite numbers: zero K, V and the query ring.
bool clear_arena(mkv_ctx *c, cudaStream_t stream)
{
    const size_t kv = (size_t)c->s.U * c->s.cap * c->s.D * c->s.es, rq = (size_t)c->s.U * c->s.R * c->s.G * c->s.D * c->s.es;
    return cudaMemsetAsync(c->base + c->L.K, 0, kv, stream) == cudaSuccess &&
           cudaMemsetAsync(c->base + c->L.V, 0, kv, stream) == cudaSuccess &&
           cudaMemsetAsync(c->base + c->L.ring_q, 0, rq, stream) == cudaSuccess;
}

mkv_status launch_step(mkv_ctx *ctx, const void *q, const void *k, const void *v, void *out, cudaStream_t stream)
{
    const DecodeArgs a = make_args(ctx, q, k, v, out);
    const cudaError_t e = ctx->kind == kKindTc ? launch_decode_tc(ctx->plan, a, stream)
                                               : launch_decode_simt(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, stream);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "decode launch failed: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    const bool ev = step_scores(ctx->t, ctx->n, ctx->steps, ctx->s.R, ctx->s.C, ctx->s.T);
    // coarse-grained eviction: the compaction follows the steps that ran the policy (the kernel itself checks the
    // device state and does nothing if no compaction is pending)
    if (ctx->s.T > 1 && ev) {
        const cudaError_t e2 = launch_compact(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, stream);
        if (e2 != cudaSuccess) return fail(ctx, MKV_CUDA, "compaction launch failed: %s", cudaGetErrorString(e2));
        ctx->launches += 1;
    }
    ctx->t += 1;
    ctx->steps += 1;
    if (!ev) ctx->n += 1;
    else if (ctx->s.T > 1) ctx->n = ctx->s.C + ctx->s.R;
    return MKV_OK;
}

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

size_t mkv_workspace_bytes(const mkv_params *p)
{
    if (!params_valid(p)) return 0;
    Shape s;
    KernelKind kind;
    if (!resolve(p, &s, &kind)) return 0;
    return make_layout(s).total;
}

mkv_status mkv_create_ex(mkv_ctx **out, const mkv_params *p)
{
    if (!out) return MKV_INVALID_ARG;
    *out = nullptr;
    if (!params_valid(p)) return MKV_INVALID_ARG;
    Shape s;
    KernelKind kind;
    if (!resolve(p, &s, &kind)) return MKV_UNSUPPORTED;
    const Layout L = make_layout(s);
    if (p->workspace) {
        if (((uintptr_t)p->workspace & 255) != 0) return MKV_INVALID_ARG;
        if (p->workspace_bytes < L.total) return MKV_OOM;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        cudaGetLastError();
        return MKV_CUDA;
    }
    mkv_ctx *c = new (std::nothrow) mkv_ctx;
    if (!c) return MKV_OOM;
    memset(c, 0, sizeof(*c));
    c->p = *p; c->s = s; c->L = L; c->kind = kind;
    if (p->workspace) {
        c->base = (char *)p->workspace;
    } else {
        void *mem = nullptr;
        if (cudaMalloc(&mem, L.total) != cudaSuccess) {
            cudaGetLastError();
            delete c;
            return MKV_OOM;
        }
        c->base = (char *)mem;
        c->owns_workspace = true;
    }
    if (kind == kKindTc) {
        const DecodeArgs a = make_args(c, nullptr, nullptr, nullptr, nullptr);
        char msg[200] = "";
        const cudaError_t e = tc_plan_create(&c->plan, a, s.tc_grid_size, p->wait_limit_cycles, msg, sizeof(msg));
        if (e != cudaSuccess) {
            cudaGetLastError();
            if (c->owns_workspace) cudaFree(c->base);
            delete c;
            return e == cudaErrorMemoryAllocation ? MKV_OOM : MKV_CUDA;
        }
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
    if (ctx->plan) tc_plan_destroy(ctx->plan);
    if (ctx->prefill_scratch.ptr) cudaFree(ctx->prefill_scratch.ptr);
    if (ctx->owns_workspace && ctx->base) cudaFree(ctx->base);
    delete ctx;
}

mkv_status mkv_prefill(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!k || !v || !q_window) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill: NULL tensor%s");
    if (prompt_len < 1 || prompt_len > (1 << 24)) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill: prompt_len out of range%s");
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_prefill: context already holds a sequence%s");
    const DecodeArgs a = make_args(ctx, nullptr, nullptr, nullptr, nullptr);
    if (!clear_arena(ctx, (cudaStream_t)stream)) return fail(ctx, MKV_CUDA, "mkv_prefill: clearing the arena failed%s");
    const cudaError_t e = run_prefill(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, k, v, q_window, prompt_len,
                                      (cudaStream_t)stream, &ctx->launches, &ctx->prefill_scratch);
    if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return fail(ctx, MKV_OOM, "mkv_prefill: no memory for scratch%s"); }
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_prefill: %s", cudaGetErrorString(e));
    const int Rw = prompt_len < ctx->s.R ? prompt_len : ctx->s.R;
    ctx->n = (prompt_len - Rw > ctx->s.C) ? ctx->s.C + Rw : prompt_len;
    ctx->t = prompt_len;
    ctx->steps = 0;
    ctx->prefilled = true;
    return MKV_OK;
}

mkv_status mkv_prefill_static(mkv_ctx *ctx, const void *k, const void *v, const void *q_window, int prompt_len, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!k || !v || !q_window) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_static: NULL tensor%s");
    if (prompt_len < 1 || prompt_len > (1 << 24)) return fail(ctx, MKV_INVALID_ARG, "mkv_prefill_static: prompt_len out of range%s");
    if (ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_prefill_static: context already holds a sequence%s");
    const int Rw = prompt_len < ctx->s.R ? prompt_len : ctx->s.R;
    const size_t need = ((size_t)Rw * ctx->s.G + 1) * (size_t)prompt_len;
    if (need > prefill_static_max_floats()) {
        snprintf(ctx->err, sizeof(ctx->err),
                 "mkv_prefill_static: one unit needs (min(R,P)*G + 1) * prompt_len = %zu floats of scratch, the fixed "
                 "array holds %zu; use mkv_prefill for this prompt", need, prefill_static_max_floats());
        return MKV_UNSUPPORTED;
    }
    const DecodeArgs a = make_args(ctx, nullptr, nullptr, nullptr, nullptr);
    if (!clear_arena(ctx, (cudaStream_t)stream)) return fail(ctx, MKV_CUDA, "mkv_prefill_static: clearing the arena failed%s");
    const cudaError_t e = run_prefill_static(a, ctx->p.dtype == MKV_DTYPE_F32, ctx->s.D, k, v, q_window, prompt_len,
                                             (cudaStream_t)stream, &ctx->launches);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_prefill_static: %s", cudaGetErrorString(e));
    ctx->n = (prompt_len - Rw > ctx->s.C) ? ctx->s.C + Rw : prompt_len;
    ctx->t = prompt_len;
    ctx->steps = 0;
    ctx->prefilled = true;
    return MKV_OK;
}

mkv_status mkv_decode_step(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *out, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (!q || !k_new || !v_new || !out) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_step: NULL tensor%s");
    if (!ctx->prefilled) return fail(ctx, MKV_BAD_STATE, "mkv_decode_step: call mkv_prefill first%s");
    if (ctx->t >= 0x7fffffffLL) return fail(ctx, MKV_UNSUPPORTED, "mkv_decode_step: position exceeds int32%s");
    return launch_step(ctx, q, k_new, v_new, out, (cudaStream_t)stream);
}

mkv_status mkv_decode_steps(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *out, int n_steps,
                            void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    if (n_steps < 0) return fail(ctx, MKV_INVALID_ARG, "mkv_decode_steps: negative n_steps%s");
    const size_t qb = (size_t)ctx->s.U * ctx->s.G * ctx->s.D * ctx->s.es, kb = (size_t)ctx->s.U * ctx->s.D * ctx->s.es;
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
    cudaStream_t s = (cudaStream_t)stream;
    const size_t qb = (size_t)ctx->s.U * ctx->s.G * ctx->s.D * ctx->s.es, kb = (size_t)ctx->s.U * ctx->s.D * ctx->s.es;
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
    const size_t upl = (size_t)ctx->p.batch * ctx->p.n_kv_heads, u0 = upl * layer;
    const Shape &s = ctx->s;
    char *b = ctx->base;
    view->K = b + ctx->L.K + u0 * s.cap * s.D * s.es;
    view->V = b + ctx->L.V + u0 * s.cap * s.D * s.es;
    view->pos = (int32_t *)(b + ctx->L.pos) + u0 * s.cap;
    view->F = (float *)(b + ctx->L.F) + u0 * s.cap;
    view->evicted_pos = (int32_t *)(b + ctx->L.evicted) + u0;
    view->ring_q = b + ctx->L.ring_q + u0 * s.R * s.G * s.D * s.es;
    view->ring_c = (float *)(b + ctx->L.ring_c) + u0 * s.R * s.G;
    view->count = ctx->n;
    view->capacity = s.cap;
    view->next_pos = ctx->t;
    return MKV_OK;
}

mkv_status mkv_sync(mkv_ctx *ctx, void *stream)
{
    if (!ctx) return MKV_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_sync: %s", cudaGetErrorString(e));
    DevState st;
    e = cudaMemcpy(&st, ctx->base + ctx->L.state, sizeof(st), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(ctx, MKV_CUDA, "mkv_sync: %s", cudaGetErrorString(e));
    if (st.err == kErrCacheOverflow)
        return fail(ctx, MKV_BAD_STATE, "a decode step found no free slot: coarse-grained eviction ran out of step%s");
    if (st.err != kErrNone) {
        char code[32];
        snprintf(code, sizeof(code), " (wait code %d)", st.err);
        return fail(ctx, MKV_DEVICE_TIMEOUT, "a device-side wait ran out of iterations%s", code);
    }
    // the device-resident state is authoritative (steps replayed from a CUDA graph advance
    // it without passing through this library); the host mirror follows it
    if (ctx->prefilled) { ctx->t = st.t; ctx->n = st.n; ctx->steps = st.steps; }
    return MKV_OK;
}

const char *mkv_last_error(const mkv_ctx *ctx) { return ctx ? ctx->err : ""; }

uint64_t mkv_launch_count(const mkv_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *mkv_kernel_name(const mkv_ctx *ctx) { return (ctx && ctx->kind == kKindTc) ? "tc" : "simt"; }

}  // extern "C"
