// Shared device-side definitions of the MorphKV decode path: argument blocks, element
// helpers and the per-unit epilogue that merges split partials, selects the eviction and
// appends the new token (Eq. 1 merge, Eq. 4-7, Algorithm 1 of the paper).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mkv {

constexpr int kMaxGroup = 16;     // largest supported GQA group size
constexpr int kFusionSum = 0;
constexpr int kFusionMax = 1;

// Device-resident step state.  Kernels read it at entry and one CTA of each launch advances it
// (the last one to finish in the CUDA-core kernel, the last one to have read it in the
// tensor-core kernel), so consecutive launches need no host-side step index.
struct DevState {
    long long t;          // absolute position of the token being decoded
    int n;                // tokens cached per unit before this step
    int steps;            // decode steps completed
    int err;              // sticky device-side error code (0 = none)
    unsigned int done;    // CTAs of the current launch that have finished
    int compact;          // coarse-grained eviction: the step that just ran scored, the cache awaits its compaction
};

// 1..99: the code of the bounded wait that gave up; kErrCacheOverflow: a step found no free slot (only possible
// when coarse-grained eviction was driven out of step, e.g. by replaying part of a period from a CUDA graph)
enum DevError { kErrNone = 0, kErrBarrierTimeout = 1, kErrCacheOverflow = 100 };

// Everything a decode kernel needs.  Passed by value as a __grid_constant__.
struct DecodeArgs {
    void *K, *V;               // [U][cap][D]
    int *pos;                  // [U][cap]
    void *ring_q;              // [U][R][G][D]
    float *ring_c;             // [U][R][G]
    const void *q, *k_new, *v_new;
    void *out;
    float *s_new;              // [U][G][cap]   scaled log2-domain logits of the new query
    float *F;                  // [U][cap]      fused score (partial, then final)
    float *part_ml;            // [U][splits][G][2]  (max, denominator) of each split
    float *part_o;             // [U][splits][G][D]  un-normalised split outputs
    int *ticket;               // [U]
    int *evicted_pos;          // [U]
    DevState *st;              // the step state this launch reads and advances
    int u0;                    // index of this launch's first unit in the context's arena (per-layer launches): the
                               // pointers above are already offset by it, tensor-map coordinates are not
    int U, G, R, C, cap, splits, fusion, T;
    int norm_current;          // 1: CURRENT normalisation - window rows are renormalised over the tokens still cached
    int Gq;                    // query heads per unit in q and out (the model's GQA ratio).  G, the group the arena
                               // and the kernels work with, is Gq rounded up to a power of two on the tensor-core path:
                               // heads Gq .. G-1 have a zero query and normaliser +inf (weight 0) and produce no output
    float scale2;              // log2(e) / sqrt(D)
    float *Fc;                 // [U][nc][cap]  tensor-core kernel with a window of nc > 1 ring chunks: the fused score of
    int nc;                    // each chunk's rows, combined by the unit's epilogue; unused (nullptr, 1) otherwise
    // Batch rows with prompts of different lengths (nullptr / unused otherwise).  The step state then counts time
    // from the longest prompt: st->t is that row's position and st->n the largest fill; row b is row_shift[b]
    // positions behind (its token has position st->t - row_shift[b]) and holds row_n[(st->steps & 1) * B + b]
    // tokens.  The fills are double-buffered by step parity because the CTA that advances the state does so while
    // other CTAs of the launch still read the current fills.  Ring slots are assigned by st->t in every row.
    int *row_n;                // [2][B]
    const int *row_shift;      // [B]
    int B, Hkv;                // unit u (of this launch) belongs to batch row (u / Hkv) % B
    float *prof;               // [U][R][cap]  stored-profile mode (nullptr otherwise): prof[r][k] is the weight, summed
                               // over the group, that the window token of ring slot r gave to the token in cache slot
                               // k when it was generated (the attention profile the paper's implementation stores
                               // beside the KV cache); the fused scores are then read from this table, not recomputed
    int n_hint;                // the host's view of st->n when the launch was enqueued (0: none).  Only used to
                               // prefetch: a stale value (steps replayed from a CUDA graph) costs time, not results
};

// Fill, position offset and policy decision of one unit on this step.
struct UnitStep {
    int n, shift;
    bool evict;
};

__device__ __forceinline__ float ldf(const float *p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float *p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float fuse(int fusion, float a, float b)
{
    return fusion == kFusionSum ? a + b : fmaxf(a, b);
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

// Ordering key of a candidate: larger key = better.  Fused scores are non-negative floats,
// whose bit patterns order like the values; among equal scores the LOWER position gets the
// larger key, so it is the one kept.  All keys of a unit are distinct.
__host__ __device__ __forceinline__ unsigned long long rank_key(unsigned int F_bits, int pos)
{
    return ((unsigned long long)F_bits << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)pos);
}

// How a unit's n cached tokens are divided among `splits` CTAs: contiguous ranges whose
// length is a multiple of `tile`.  Returns the per-split length; *active = splits with work.
__host__ __device__ inline int split_len(int n, int splits, int tile, int *active)
{
    const int tiles = (n + tile - 1) / tile;
    const int per = ((tiles + splits - 1) / splits) * tile;
    *active = per > 0 ? (n + per - 1) / per : 0;
    return per;
}

// True when this step must evict: after the new token joins, the tokens outside the window
// of min(R, t+1) recent ones exceed C (Eq. 7 keeps the cache at C + R).
__host__ __device__ inline bool step_evicts(long long t, int n, int R, int C)
{
    const long long win = (t + 1 < (long long)R) ? t + 1 : (long long)R;
    return (long long)n + 1 - win > (long long)C;
}

// True when this step runs the policy (scores and evicts).  With evict_interval T > 1 (coarse-grained
// eviction appendix) that is every T-th decode step only, and the step then appends like any other:
// a separate compaction launch drops everything beyond the top C afterwards.
__host__ __device__ inline bool step_scores(long long t, int n, int steps, int R, int C, int T)
{
    if (T > 1 && (steps + 1) % T != 0) return false;
    return step_evicts(t, n, R, C);
}

constexpr int kFinalizeSmemFloats = 4 * kMaxGroup + 3 * 32 + 128;

// `evict` is the decision for the uniform state (t, n); rows of different lengths take their own.
__device__ __forceinline__ UnitStep unit_step(const DecodeArgs &a, int u, long long t, int n, int steps, bool evict)
{
    UnitStep s;
    s.n = n; s.shift = 0; s.evict = evict;
    if (a.row_n != nullptr) {
        const int b = (u / a.Hkv) % a.B;
        s.n = a.row_n[(steps & 1) * a.B + b];
        s.shift = a.row_shift[b];
        s.evict = step_scores(t - s.shift, s.n, steps, a.R, a.C, a.T);
    }
    return s;
}

// The step state after this launch (called by one thread, once per launch, after every CTA has read the state).
__device__ __forceinline__ void advance_state(const DecodeArgs &a, long long t, int n, int steps, bool evict)
{
    int n_next = (evict && a.T == 1) ? n : n + 1;
    if (a.row_n != nullptr) {      // every row appends or evicts by its own fill; the uniform fill is the largest
        n_next = 0;
        const int *cur = a.row_n + (steps & 1) * a.B;
        int *nxt = a.row_n + ((steps + 1) & 1) * a.B;
        for (int b = 0; b < a.B; ++b) {
            const int nb = cur[b];
            const int v = step_scores(t - a.row_shift[b], nb, steps, a.R, a.C, a.T) ? nb : nb + 1;
            nxt[b] = v;
            n_next = v > n_next ? v : n_next;
        }
    }
    a.st->t = t + 1;
    a.st->n = n_next;
    a.st->compact = (evict && a.T > 1) ? 1 : 0;
    a.st->steps = steps + 1;
    a.st->done = 0;
}


// barrier over the `nthr` threads that run an epilogue together (id 0 with the whole CTA is
// __syncthreads; warp-specialised kernels give each compute group its own id)
__device__ __forceinline__ void group_sync(int bar_id, int nthr)
{
    // barrier.sync without .aligned (bar.sync is the aligned form): the lanes of a warp may reach this
    // point on different paths, e.g. straight after an `if (tid < k)` block, and each counts for itself
    asm volatile("barrier.sync %0, %1;" ::"r"(bar_id), "r"(nthr) : "memory");
}

// CURRENT normalisation (the reading of Eq. 4 in which a window row's weights are taken over the tokens that are
// still cached): the token in `e_slot` is about to be evicted, so every window row loses the weight w it had on it
// and its log2-domain normaliser becomes c + log2(1 - w); the surviving weights of the row grow by 1 / (1 - w).
// Rows of the ring: the row `rs_new` is being replaced by the new query, whose normaliser is cnew[g] (shared memory,
// updated in place) and whose logits on the evicted key are in s_new; the other rows' logits are recomputed from
// the stored queries.  `krow` is scratch for D floats.  Called by the whole group before the evicted slot's K row
// is overwritten.
template <typename T, int D>
__device__ void renormalise_after_eviction(const DecodeArgs &a, int u, int e_slot, int rs_new, float *cnew, float *krow,
                                           int tid, int nthr, int bar_id)
{
    const int G = a.G;
    const T *Ke = static_cast<const T *>(a.K) + ((size_t)u * a.cap + e_slot) * D;
    for (int i = tid; i < D; i += nthr) krow[i] = ldf(Ke + i);
    group_sync(bar_id, nthr);
    const T *ring_q = static_cast<const T *>(a.ring_q) + (size_t)u * a.R * G * D;
    float *ring_c = a.ring_c + (size_t)u * a.R * G;
    for (int row = tid; row < a.R * G; row += nthr) {
        const int rslot = row / G, g = row % G;
        float c, s;
        if (rslot == rs_new) {
            c = cnew[g];
            s = __ldcg(a.s_new + ((size_t)u * G + g) * a.cap + e_slot);
        } else {
            c = ring_c[row];
            s = 0.f;
            if (c < INFINITY) {
                const T *qr = ring_q + (size_t)row * D;
                float acc = 0.f;
                for (int i = 0; i < D; ++i) acc += ldf(qr + i) * krow[i];
                s = acc * a.scale2;
            }
        }
        if (c < INFINITY) {
            const float w = exp2f(s - c);
            c += log2f(fmaxf(1.f - w, 1e-30f));
            if (rslot == rs_new) cnew[g] = c; else ring_c[row] = c;
        }
    }
    group_sync(bar_id, nthr);
}


// Per-unit epilogue, run by the group of threads that finished a unit last (`tid` in
// [0, nthr), nthr a multiple of 32, all of them synchronising on barrier `bar_id`).  Data
// written by other CTAs is read with ld.global.cg so that no stale L1 line can be used.
// `sm` needs kFinalizeSmemFloats floats of shared memory, 8-byte aligned.  GT is the GQA
// group size when known at compile time (0: use a.G); it lets the loads of a round be
// issued together.  Loads are batched so that the whole epilogue costs a handful of L2
// round trips.
// PROF: the caller may be serving the stored-profile mode (a.prof); compiled out otherwise.
template <typename T, int D, int GT, bool PROF = false>
__device__ void finalize_unit(const DecodeArgs &a, int u, long long t, int n, int active, bool evict, float *sm,
                              int tid, int nthr, int bar_id, int shift = 0)
{
    const int lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const int G = GT > 0 ? GT : a.G;
    constexpr int GU = GT > 0 ? GT : 1;    // unroll width of the per-head loads
    float *s_self = sm, *mfin = sm + kMaxGroup, *lfin = sm + 2 * kMaxGroup, *cnew = sm + 3 * kMaxGroup;
    unsigned long long *red_key = reinterpret_cast<unsigned long long *>(sm + 4 * kMaxGroup);  // [32]
    int *red_slot = reinterpret_cast<int *>(sm + 4 * kMaxGroup + 64);                          // [32]

    const int Gq = a.Gq;
    const T *q = static_cast<const T *>(a.q) + (size_t)u * Gq * D;
    const T *kn = static_cast<const T *>(a.k_new) + (size_t)u * D;
    const T *vn = static_cast<const T *>(a.v_new) + (size_t)u * D;
    const float *pml = a.part_ml + (size_t)u * a.splits * G * 2;
    const float *po = a.part_o + (size_t)u * a.splits * G * D;

    // the new token attends to itself (self-inclusive Eq. 1): one more logit per head
    for (int g = warp; g < G; g += nwarp) {
        float acc = 0.f;
        if (g < Gq)
            for (int i = lane; i < D; i += 32) acc += ldf(q + g * D + i) * ldf(kn + i);
        acc = warp_sum(acc);
        if (lane == 0) s_self[g] = acc * a.scale2;
    }
    group_sync(bar_id, nthr);
    if (tid < G) {
        // two passes over the partial (max, denominator) pairs, eight loads in flight at a time
        float m = s_self[tid];
        for (int sp0 = 0; sp0 < active; sp0 += 8) {
            float pm[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) pm[i] = sp0 + i < active ? __ldcg(pml + ((sp0 + i) * G + tid) * 2) : -INFINITY;
#pragma unroll
            for (int i = 0; i < 8; ++i) m = fmaxf(m, pm[i]);
        }
        float l = exp2f(s_self[tid] - m);
        for (int sp0 = 0; sp0 < active; sp0 += 8) {
            float pm[8], pl[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool ok = sp0 + i < active;
                pm[i] = ok ? __ldcg(pml + ((sp0 + i) * G + tid) * 2) : -INFINITY;
                pl[i] = ok ? __ldcg(pml + ((sp0 + i) * G + tid) * 2 + 1) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) l += pl[i] * exp2f(pm[i] - m);
        }
        mfin[tid] = m;
        lfin[tid] = l;
        cnew[tid] = tid < Gq ? m + log2f(l) : INFINITY;
    }
    group_sync(bar_id, nthr);
    T *out = static_cast<T *>(a.out) + (size_t)u * Gq * D;
    for (int idx = tid; idx < Gq * D; idx += nthr) {
        const int g = idx / D, dd = idx % D;
        const float m = mfin[g];
        float o = exp2f(s_self[g] - m) * ldf(vn + dd);
        for (int sp0 = 0; sp0 < active; sp0 += 8) {
            float pv[8], pm[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool ok = sp0 + i < active;
                pv[i] = ok ? __ldcg(po + ((sp0 + i) * G + g) * D + dd) : 0.f;
                pm[i] = ok ? __ldcg(pml + ((sp0 + i) * G + g) * 2) : -INFINITY;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) o += pv[i] * exp2f(pm[i] - m);
        }
        stf(out + idx, o / lfin[g]);
    }

    // Algorithm 1 / Eq. 7: add the new row's term to the fused scores, evict the minimum
    int *pos = a.pos + (size_t)u * a.cap;
    float *F = a.F + (size_t)u * a.cap;
    int e_slot = n, e_pos = -1;
    // stored-profile mode: the new token's row of the table is written on every step, policy or not
    float *prof_row = nullptr;
    if constexpr (PROF) prof_row = a.prof ? a.prof + ((size_t)u * a.R + (int)(t % a.R)) * a.cap : nullptr;
    if (PROF && prof_row != nullptr && !evict) {
        const float *sn = a.s_new + (size_t)u * G * a.cap;
        for (int k = tid; k < n; k += nthr) {
            float s = 0.f;
            for (int g = 0; g < G; ++g) s += exp2f(__ldcg(sn + (size_t)g * a.cap + k) - cnew[g]);
            prof_row[k] = s;
        }
    }
    if (evict) {
        const float *sn = a.s_new + (size_t)u * G * a.cap;
        const long long thr = t - shift - a.R;        // positions are the row's own; ring slots follow t
        unsigned long long best = ~0ull;
        int bslot = -1;
        // four slots per thread and round, all their loads in flight together
        for (int kb = tid; kb < n; kb += 4 * nthr) {
            int p[4];
            float f0[4], s[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int k = kb + b * nthr;
                p[b] = k < n ? pos[k] : 0x7fffffff;
                f0[b] = k < n ? __ldcg(F + k) : 0.f;
                s[b] = 0.f;
            }
            for (int g0 = 0; g0 < G; g0 += GU) {
                float x[GU][4];
#pragma unroll
                for (int gi = 0; gi < GU; ++gi)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int k = kb + b * nthr;
                        x[gi][b] = k < n ? __ldcg(sn + (size_t)(g0 + gi) * a.cap + k) : -INFINITY;
                    }
#pragma unroll
                for (int gi = 0; gi < GU; ++gi)
#pragma unroll
                    for (int b = 0; b < 4; ++b) s[b] += exp2f(x[gi][b] - cnew[g0 + gi]);
            }
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int k = kb + b * nthr;
                if (k >= n) continue;
                if (PROF && prof_row != nullptr) prof_row[k] = s[b];
                if ((long long)p[b] <= thr) {
                    const float f = fuse(a.fusion, f0[b], s[b]);
                    F[k] = f;
                    const unsigned long long key = rank_key(__float_as_uint(f), p[b]);
                    if (key < best) { best = key; bslot = k; }
                } else {
                    F[k] = -1.f;   // window slot: not a candidate
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
            const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
            if (ok < best) { best = ok; bslot = os; }
        }
        if (lane == 0) { red_key[warp] = best; red_slot[warp] = bslot; }
        group_sync(bar_id, nthr);
        if (warp == 0) {
            best = lane < nwarp ? red_key[lane] : ~0ull;
            bslot = lane < nwarp ? red_slot[lane] : -1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
                const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
                if (ok < best) { best = ok; bslot = os; }
            }
            if (lane == 0) red_slot[0] = bslot;
        }
        group_sync(bar_id, nthr);
        e_slot = red_slot[0];
        e_pos = pos[e_slot];
        group_sync(bar_id, nthr);
        if (a.T > 1) {          // coarse-grained eviction: append now, the compaction launch evicts
            e_slot = n;
            e_pos = -1;
            if (tid == 0 && n < a.cap) F[n] = -1.f;
        } else if (a.norm_current) {
            renormalise_after_eviction<T, D>(a, u, e_slot, (int)(t % a.R), cnew, sm + 4 * kMaxGroup + 3 * 32, tid, nthr, bar_id);
        }
    }

    if (e_slot >= a.cap) {      // no free slot: refuse to write beyond the unit's rows
        if (tid == 0) { atomicCAS(&a.st->err, 0, (int)kErrCacheOverflow); a.ticket[u] = 0; }
        return;
    }
    // Eq. 7 update: the freed (or next free) slot takes the new token; the ring row of the
    // token that left the window takes the new query and its soft-max normaliser
    T *Kd = static_cast<T *>(a.K) + ((size_t)u * a.cap + e_slot) * D;
    T *Vd = static_cast<T *>(a.V) + ((size_t)u * a.cap + e_slot) * D;
    for (int i = tid; i < D; i += nthr) { Kd[i] = kn[i]; Vd[i] = vn[i]; }
    const int rs = (int)(t % a.R);
    T *rq = static_cast<T *>(a.ring_q) + ((size_t)u * a.R + rs) * G * D;
    for (int i = tid; i < G * D; i += nthr) stf(rq + i, i < Gq * D ? ldf(q + i) : 0.f);
    if (tid < G) a.ring_c[((size_t)u * a.R + rs) * G + tid] = cnew[tid];
    if (PROF && a.prof != nullptr) {
        // the slot the new token takes: no older window token ever attended to it; the new token's weight on itself
        float self_w = 0.f;
        for (int g = 0; g < G; ++g) self_w += exp2f(s_self[g] - cnew[g]);
        float *col = a.prof + (size_t)u * a.R * a.cap + e_slot;
        for (int r = tid; r < a.R; r += nthr) col[(size_t)r * a.cap] = r == rs ? self_w : 0.f;
    }
    if (tid == 0) {
        pos[e_slot] = (int)(t - shift);
        a.evicted_pos[u] = e_pos;
        a.ticket[u] = 0;
    }
}

// Last action of every CTA of a decode launch: the CTA that finishes last advances the
// device-resident step state.  Must be called by all CTAs, after all their other work,
// so that no CTA can still be about to read the state when it changes.
__device__ __forceinline__ void finish_cta(const DecodeArgs &a, long long t, int n, bool evict)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int total = gridDim.x * gridDim.y * gridDim.z;
        if (atomicAdd(&a.st->done, 1u) == total - 1) {
            advance_state(a, t, n, a.st->steps, evict);
            __threadfence();
        }
    }
}

}  // namespace mkv
