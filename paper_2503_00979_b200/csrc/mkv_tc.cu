// Tensor-core decode kernel for sm_100a: bf16, head_dim 128, GQA group in {1,2,4,8,16}.  Up to 256
// ring rows (R*G, padded to a multiple of 32) are one MMA operand; a larger window is cut into
// chunks of equal width and a unit is then scheduled once per chunk (template parameter MC, see the
// kernel's prologue).
//
// The 128-key tiles of all units' caches form one sequence that is cut into equal contiguous
// ranges, one per persistent, warp-specialised CTA; a work item is the run of a unit's tiles
// inside a CTA's range.  Per tile the K rows feed the scoring contraction and the V rows the
// attention output; both are read from HBM exactly once.
//   warp 0       TMA producer of the unit's recent-query ring (once per unit) and of K tiles
//                (cp.async.bulk.tensor, 128-byte swizzle) into a short ring of 32 KB stages.
//   warp 1       writes the new query over the ring row that leaves the window, then issues
//                tcgen05.mma: S^T[128 keys x R*G rows] = K_tile . Q^T, fp32 accumulators in
//                TMEM (one key per TMEM lane), up to four accumulator buffers, so K stages are
//                released as soon as their MMA has run.
//   warp 2       TMA producer of V tiles into their own ring of stages.
//   warps 3-10   two compute groups of four warps; tiles alternate between the groups and
//                each warp owns the 32 keys of its TMEM lane quarter.  Per tile: tcgen05.ld of
//                a key's R*G logits, frozen soft-max weights exp2(s*scale - c_row), GQA group
//                sum, window fusion (Eq. 4-6, Algorithm 1); then the new row's soft-max is
//                continued online (running max per head, rescale) and P.V for the warp's keys
//                runs on mma.sync with P split in two bf16 terms (Eq. 1).  Compute warps only
//                meet at mbarriers; when a unit's tiles in this CTA are done each warp leaves
//                its partial (m, l, O) in shared memory and goes on with the next unit.
//   warps 11-14  epilogue group: merges the eight warp partials of a unit; if the unit spans
//                several CTAs it publishes the CTA's partial and an atomic ticket (no waiting)
//                elects the last CTA; that group merges, writes the output, adds the new row's
//                term to the fused scores, evicts and appends (Eq. 7).  Compute never stalls on it.
// Every mbarrier wait is bounded; a wait that runs out sets a device error flag and the CTA
// drains and exits.  Warp-collective .aligned instructions (ldmatrix, mma.sync, tcgen05.ld)
// are only reached with the whole warp converged: the code before them is branch-free or
// ends in a warp-level sync.
#include <cuda.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "mkv_common.cuh"
#include "mkv_kernels.h"
#include "mkv_schedule.h"
#include "mkv_sm100.cuh"

namespace mkv {

namespace {

constexpr int kComputeGroups = 2;
constexpr int kMaxComputeWarps = 4 * kComputeGroups;
// 3 service warps + 4 per compute group + 4 epilogue warps
__host__ __device__ constexpr int tc_threads(int ng) { return 32 * (3 + 4 * ng + 4); }
constexpr int kFirstComputeWarp = 3;
constexpr int kFinFloats = 4 * kMaxGroup + 128 + 256 + 64 + 32 + 8;   // epilogue scratch of finalize_fast
// epilogue group: finalize scratch, flag, merged (m, l), per-warp scale factors
constexpr int kEpiFloats = kFinFloats + 8 + 2 * kMaxGroup + kMaxComputeWarps * kMaxGroup;

struct TcGeom {
    int rgpad;          // ring rows of one chunk, padded to a multiple of 32 (MMA N)
    int nc;             // ring chunks (1 unless the window has more than 256 rows)
    int sk, sv;         // K stages, V stages
    int ng;             // compute groups; tile T belongs to group T % ng
    int nb;             // TMEM accumulator buffers (a multiple of ng)
    int tmem_cols;      // allocated TMEM columns (power of two)
    int grid;
    int smem_bytes;
    long long wait_cycles;   // limit of every device-side wait, in clock64 ticks
    int prefetch_tiles;      // K and V tiles a CTA asks into L2 before it waits for the previous grid (0: none)
};

struct SmemLayout {
    int q, kst, vst, wbuf, wml, negc, stw, epi, bars, total;
};

__host__ __device__ inline SmemLayout tc_smem_layout(const TcGeom &g, int G)
{
    SmemLayout L;
    int o = 0;
    L.q = o; o += g.rgpad * 256;
    L.kst = o; o += g.sk * kStageBytes;
    L.vst = o; o += g.sv * kStageBytes;
    const int ncw = 4 * g.ng;                         // compute warps
    L.wbuf = o; o += ncw * G * kD * 4;                // a warp's un-normalised output O[g][d] of a finished unit
    L.wml = o; o += ncw * 2 * kMaxGroup * 4;          // ... and its (max, denominator) per head
    L.negc = o; o += ncw * g.rgpad * 4;               // negated ring normalisers, one copy per compute warp
    L.stw = o; o += ncw * (G * 32 + 2 * kMaxGroup) * 4; // per warp: kept logits of one tile, rescale factors, reference
    L.epi = o; o += kEpiFloats * 4;
    o = (o + 15) & ~15;
    L.bars = o; o += 8 * 64;
    L.total = o;
    return L;
}

// ---------------------------------------------------------------- schedule shared by all roles: mkv_schedule.h
static_assert(kSchedTile == kTile, "the schedule and the kernel must agree on the tile");

// position in a ring of n slots (stage or accumulator buffer) and the parity of the lap,
// advanced without divisions
struct RingPos {
    int idx, lap;
    __device__ RingPos(int start, int n) : idx(start % n), lap((start / n) & 1) {}
    __device__ __forceinline__ void step(int by, int n)
    {
        idx += by;
        while (idx >= n) { idx -= n; lap ^= 1; }
    }
};

// Per-unit epilogue for a compute group of 128 threads (same result as finalize_unit): merge the
// segments' partials, write the attention output, add the new row's term to the fused scores,
// evict the minimum, append (Eq. 1 merge, Eq. 4-7).  All loads of a phase are issued together, so
// the whole epilogue costs a few L2 round trips.  Requires nseg <= 8 and nseg*G*2 <= 256.
// LOCAL: the single partial is this CTA's own: l_o[g] is the thread's column of the merged output,
// l_ml [G][2] sits in shared memory.
template <int G, bool LOCAL>
__device__ void finalize_fast(const DecodeArgs &a, int u, long long t, int n, int nseg, bool evict, float *sm, int tid,
                              int bar_id, const float (&l_o)[G], const float *l_ml, int shift)
{
    constexpr int NT_ = kGroupThreads;
    const int lane = tid & 31, warp = tid >> 5;
    float *s_self = sm, *mfin = sm + kMaxGroup, *lfin = sm + 2 * kMaxGroup, *cnew = sm + 3 * kMaxGroup;
    float *vsm = sm + 4 * kMaxGroup;                       // [128] new value row as floats
    float *pml_s = vsm + 128;                              // [nseg][G][2]
    unsigned long long *red_key = reinterpret_cast<unsigned long long *>(pml_s + 256);   // [32]
    int *red_slot = reinterpret_cast<int *>(pml_s + 256 + 64);                           // [32]

    const int Gq = a.Gq;      // heads Gq .. G-1 are padding: zero query, normaliser +inf, no output
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(a.q) + (size_t)u * Gq * kD;
    const __nv_bfloat16 *kn = static_cast<const __nv_bfloat16 *>(a.k_new) + (size_t)u * kD;
    const __nv_bfloat16 *vn = static_cast<const __nv_bfloat16 *>(a.v_new) + (size_t)u * kD;
    const float *pml = a.part_ml + (size_t)u * a.splits * G * 2;
    const float *po = a.part_o + (size_t)u * a.splits * G * kD;

    // ---- phase A: every load that does not depend on another one
    constexpr int QCH = (G * 16 + NT_ - 1) / NT_;          // 16-byte chunks of q per thread
    uint4 qv[QCH], kv[QCH];
#pragma unroll
    for (int i = 0; i < QCH; ++i) {
        const int c = tid + i * NT_;
        if (c < G * 16) {
            qv[i] = c < Gq * 16 ? reinterpret_cast<const uint4 *>(q)[c] : make_uint4(0, 0, 0, 0);
            kv[i] = reinterpret_cast<const uint4 *>(kn)[c & 15];
        }
    }
    uint4 vv = make_uint4(0, 0, 0, 0);
    if (tid < 16) vv = reinterpret_cast<const uint4 *>(vn)[tid];
    for (int i = tid; i < nseg * G * 2; i += NT_) pml_s[i] = LOCAL ? l_ml[i] : __ldcg(pml + i);
    float pov[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int sp = 0; sp < 8; ++sp)
            pov[g][sp] = sp < nseg ? (LOCAL ? l_o[g] : __ldcg(po + (sp * G + g) * kD + tid)) : 0.f;

    // self logit: 8-element partial dots, reduced over the 16 threads that share a head
#pragma unroll
    for (int i = 0; i < QCH; ++i) {
        const int c = tid + i * NT_;
        float acc = 0.f;
        if (c < G * 16) {
            const uint32_t *qa = reinterpret_cast<const uint32_t *>(&qv[i]), *ka = reinterpret_cast<const uint32_t *>(&kv[i]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc += __uint_as_float(qa[e] << 16) * __uint_as_float(ka[e] << 16);
                acc += __uint_as_float(qa[e] & 0xffff0000u) * __uint_as_float(ka[e] & 0xffff0000u);
            }
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (c < G * 16 && (c & 15) == 0) s_self[c >> 4] = acc * a.scale2;
    }
    if (tid < 16) {
        const uint32_t *va = reinterpret_cast<const uint32_t *>(&vv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            vsm[tid * 8 + 2 * e] = __uint_as_float(va[e] << 16);
            vsm[tid * 8 + 2 * e + 1] = __uint_as_float(va[e] & 0xffff0000u);
        }
    }
    group_sync(bar_id, NT_);

    // ---- phase B: merged soft-max statistics, attention output
    if (tid < G) {
        float m = s_self[tid];
        for (int sp = 0; sp < nseg; ++sp) m = fmaxf(m, pml_s[(sp * G + tid) * 2]);
        float l = exp2f(s_self[tid] - m);
        for (int sp = 0; sp < nseg; ++sp) l += pml_s[(sp * G + tid) * 2 + 1] * exp2f(pml_s[(sp * G + tid) * 2] - m);
        mfin[tid] = m;
        lfin[tid] = l;
        cnew[tid] = tid < Gq ? m + log2f(l) : INFINITY;
    }
    group_sync(bar_id, NT_);
    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(a.out) + (size_t)u * Gq * kD;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float m = mfin[g];
        float o = exp2f(s_self[g] - m) * vsm[tid];
#pragma unroll
        for (int sp = 0; sp < 8; ++sp)
            if (sp < nseg) o += pov[g][sp] * exp2f(pml_s[(sp * G + g) * 2] - m);
        if (g < Gq) out[g * kD + tid] = __float2bfloat16_rn(o / lfin[g]);
    }

    // ---- phase C: final fused scores and the eviction (Algorithm 1 / Eq. 7)
    int *pos = a.pos + (size_t)u * a.cap;
    float *F = a.F + (size_t)u * a.cap;
    int e_slot = n, e_pos = -1;
    if (!evict) {
        // no selection on this step (cache still filling, or between two runs of a coarse-grained policy):
        // the new token takes the next free slot
        if (tid == 0 && n < a.cap) F[n] = -1.f;
    } else {
        const float *sn = a.s_new + (size_t)u * G * a.cap;
        const long long thr = t - shift - a.R;        // positions are the row's own; ring slots follow t
        float cn[G];
#pragma unroll
        for (int g = 0; g < G; ++g) cn[g] = cnew[g];
        unsigned long long best = ~0ull;
        int bslot = -1;
        constexpr int B = 8;          // slots per thread and round, all their loads in flight together
        for (int kb = tid; kb < n; kb += B * NT_) {
            int p[B];
            float f0[B], x[G][B];
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int k = kb + b * NT_;
                p[b] = k < n ? pos[k] : 0x7fffffff;
                f0[b] = k < n ? __ldcg(F + k) : 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) x[g][b] = k < n ? __ldcg(sn + (size_t)g * a.cap + k) : -INFINITY;
            }
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int k = kb + b * NT_;
                if (k >= n) continue;
                if ((long long)p[b] <= thr) {
                    float s = 0.f;
#pragma unroll
                    for (int g = 0; g < G; ++g) s += exp2f(x[g][b] - cn[g]);
                    const float f = fuse(a.fusion, f0[b], s);
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
        group_sync(bar_id, NT_);
        best = red_key[0]; bslot = red_slot[0];
#pragma unroll
        for (int w = 1; w < NT_ / 32; ++w)
            if (red_key[w] < best) { best = red_key[w]; bslot = red_slot[w]; }
        e_slot = bslot;
        e_pos = (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull));   // the rank key carries the position
        if (a.T > 1) {
            // coarse-grained eviction (append now, the compaction launch evicts): the new token takes the
            // next free slot and is not a candidate
            e_slot = n;
            e_pos = -1;
            if (tid == 0 && n < a.cap) F[n] = -1.f;
        } else if (a.norm_current) {
            // vsm (the new value row as floats) was last read for the attention output: free to hold the evicted key
            renormalise_after_eviction<__nv_bfloat16, kD>(a, u, e_slot, (int)(t % a.R), cnew, vsm, tid, NT_, bar_id);
        }
    }

    if (e_slot >= a.cap) {      // no free slot: refuse to write beyond the unit's rows
        if (tid == 0) { atomicCAS(&a.st->err, 0, (int)kErrCacheOverflow); a.ticket[u] = 0; }
        return;
    }
    // ---- phase D: Eq. 7 update from the registers loaded in phase A
    __nv_bfloat16 *Kd = static_cast<__nv_bfloat16 *>(a.K) + ((size_t)u * a.cap + e_slot) * kD;
    __nv_bfloat16 *Vd = static_cast<__nv_bfloat16 *>(a.V) + ((size_t)u * a.cap + e_slot) * kD;
    if (tid < 16) {
        reinterpret_cast<uint4 *>(Kd)[tid] = kv[0];
        reinterpret_cast<uint4 *>(Vd)[tid] = vv;
    }
    const int rs = (int)(t % a.R);
    __nv_bfloat16 *rq = static_cast<__nv_bfloat16 *>(a.ring_q) + ((size_t)u * a.R + rs) * G * kD;
#pragma unroll
    for (int i = 0; i < QCH; ++i) {
        const int c = tid + i * NT_;
        if (c < G * 16) reinterpret_cast<uint4 *>(rq)[c] = qv[i];
    }
    if (tid < G) a.ring_c[((size_t)u * a.R + rs) * G + tid] = cnew[tid];
    if (tid == 0) {
        pos[e_slot] = (int)(t - shift);
        a.evicted_pos[u] = e_pos;
        a.ticket[u] = 0;
    }
}

// MC: the window is cut into ring chunks.  RAGGED: the batch rows have their own fills and position offsets
// (DecodeArgs::row_n); compiled separately so that the uniform kernel carries none of it.
template <int G, int FUSION, int NG, bool MC, bool RAGGED>
__global__ void __launch_bounds__(tc_threads(NG), 1)
decode_tc_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ TcGeom geo)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // the swizzled operand tiles need a 1024-byte aligned base; the launch asks for 1 KB of slack
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const SmemLayout L = tc_smem_layout(geo, G);
    const int SK = geo.sk, SV = geo.sv, NB = geo.nb, RGP = geo.rgpad;
    const long long WL = geo.wait_cycles;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t q_addr = sbase + L.q, kst_addr = sbase + L.kst, vst_addr = sbase + L.vst;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    const uint32_t bar_kfull = smem_u32(bars), bar_kempty = smem_u32(bars + 4);
    const uint32_t bar_vfull = smem_u32(bars + 8), bar_vempty = smem_u32(bars + 16);
    const uint32_t bar_tfull = smem_u32(bars + 24), bar_tempty = smem_u32(bars + 32);
    const uint32_t bar_qfull = smem_u32(bars + 40), bar_qempty = smem_u32(bars + 41);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 42);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 43);
    const uint32_t bar_udone = smem_u32(bars + 44);                    // all compute warps have left their partial of a unit
    const uint32_t bar_pfree = smem_u32(bars + 48);                    // [8] a compute warp's partial has been read

    // The tensor maps (kernel parameters) are fetched while the barriers and TMEM are set up.
    if (tid == 0) { prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); }
    if (tid == 64) prefetch_tensormap(&tmV);

    if (tid == 0) {
        for (int s = 0; s < SK; ++s) { mbar_init(bar_kfull + 8 * s, 1); mbar_init(bar_kempty + 8 * s, 1); }
        for (int s = 0; s < SV; ++s) { mbar_init(bar_vfull + 8 * s, 1); mbar_init(bar_vempty + 8 * s, 4); }
        for (int b = 0; b < NB; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
        mbar_init(bar_qfull, 1);
        mbar_init(bar_qempty, 1);
        mbar_init(bar_udone, 4 * NG);
        for (int i = 0; i < 4 * NG; ++i) mbar_init(bar_pfree + 8 * i, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), (uint32_t)geo.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Programmatic dependent launch: this grid may have been started while the grid before it in the stream was
    // still draining (a CTA gets an SM as soon as that grid's CTA there has exited), so everything above ran
    // early.  Nothing that grid wrote - step state, cache rows, query ring - is read before this wait, which
    // returns once that grid has completed and its memory operations are visible.  The next grid in the stream is
    // released at once: it parks at the same wait.
    // While the grid before this one drains (its last CTAs are in their epilogues, a chain of latencies that leaves
    // DRAM idle), this CTA asks for the first tiles of its range to be brought into L2.  A prefetch delivers no data
    // to the SM, so it may run before the wait below: rows that the previous grid's epilogues still overwrite are
    // updated in L2, which is where the loads after the wait read them.  The range is computed from the host's
    // view of the fill; if that is stale the wrong lines are prefetched and nothing else happens.  (Not in the
    // chunked-window and ragged instantiations, whose first items depend on state read after the wait.)
    if constexpr (!MC && !RAGGED) {
        if ((tid == 0 || tid == 64) && a.n_hint > 0 && geo.prefetch_tiles > 0) {
            const CUtensorMap *pm = tid == 0 ? &tmK : &tmV;
            Walk w(a.U, a.n_hint, (int)gridDim.x, (int)blockIdx.x);
            Item x;
            int left = geo.prefetch_tiles;
            while (left > 0 && w.next(x)) {
                for (int j = 0; j < x.nk && left > 0; ++j, --left) {
                    tma_prefetch_l2_3d(pm, 0, (x.tile0 + j) * kTile, a.u0 + x.unit);
                    tma_prefetch_l2_3d(pm, 64, (x.tile0 + j) * kTile, a.u0 + x.unit);
                }
                w.advance(x);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long t = a.st->t;
    const int n = a.st->n;
    const int steps_done = a.st->steps;
    __syncthreads();

    const bool evict = step_scores(t, n, steps_done, a.R, a.C, a.T);
    const int rs_new = (int)(t % a.R);
    // MC (a window of more than 256 ring rows): the ring is cut into geo.nc chunks of RGP rows = RGP / G ring
    // slots, and the schedule walks U * nc "virtual units": virtual unit v is chunk v % nc of unit v / nc.  The
    // chunk that holds the slot of the new query (the main chunk) does everything a unit does otherwise; the
    // other chunks only score their rows against the unit's keys, into their own slab of a.Fc.  On a step that
    // does not run the policy only the main chunks are walked.
    // Stored-profile mode (a.prof, served by this instantiation whatever the window's size): the fused scores of the
    // window rows come from the table (written into a.F by a launch before this one), so no chunk is scored here and
    // only the main chunk, which attends, is walked; the unit's epilogue keeps the table up to date.
    const bool stored = MC && a.prof != nullptr;
    const int NCe = MC ? ((evict && !stored) ? geo.nc : 1) : 1;  // chunks walked per unit on this step
    const int c_main = MC ? rs_new / (RGP / G) : 0;
    const int rs_loc = MC ? rs_new - c_main * (RGP / G) : rs_new;  // the new query's slot inside its chunk
    // Every thread of this CTA holds its copy of the step state (the barrier above orders their reads
    // before this point), so the CTA can be counted now: the last CTA of the launch to get here advances
    // the state for the next launch while the tiles stream, instead of at the tail of the kernel.
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(&a.st->done, 1u) == gridDim.x - 1) {
            if constexpr (RAGGED) {
                advance_state(a, t, n, steps_done, evict);
            } else {
                a.st->t = t + 1;
                a.st->n = (evict && a.T == 1) ? n : n + 1;
                a.st->compact = (evict && a.T > 1) ? 1 : 0;
                a.st->steps = steps_done + 1;
                a.st->done = 0;
            }
        }
    }

    if (warp == 0) {
        // ------------------------------------------------ TMA producer: query ring and K tiles (one lane)
        if (lane == 0) {
            Walk w(a.U * NCe, n, (int)gridDim.x, (int)blockIdx.x);
            Item x;
            int issued = 0, rings = 0;
            bool ok = true;
            RingPos rk(0, SK);
            const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
            while (ok && w.next(x)) {
                ok = mbar_wait(bar_qempty, (uint32_t)((w.nitems & 1) ^ 1), abort_flag, kWaitQEmpty, WL);
                if (!ok) break;
                const int u = MC ? x.unit / NCe : x.unit;
                const int qrow = MC ? (NCe == 1 ? c_main : x.unit - u * NCe) * RGP : 0;   // rows past R*G read as zero
                mbar_expect_tx(bar_qfull, (uint32_t)(RGP * 256));
                tma_load_3d(q_addr, &tmQ, 0, qrow, a.u0 + u, bar_qfull, pol_keep);
                tma_load_3d(q_addr + RGP * 128, &tmQ, 64, qrow, a.u0 + u, bar_qfull, pol_keep);
                ++rings;
                for (int j = 0; j < x.nk && ok; ++j, rk.step(1, SK)) {
                    const int T = w.T0 + j, s = rk.idx;
                    ok = mbar_wait(bar_kempty + 8 * s, (uint32_t)(rk.lap ^ 1), abort_flag, kWaitKEmpty, WL);
                    if (!ok) break;
                    const int row = (x.tile0 + j) * kTile;
                    mbar_expect_tx(bar_kfull + 8 * s, kStageBytes);
                    tma_load_3d(kst_addr + s * kStageBytes, &tmK, 0, row, a.u0 + u, bar_kfull + 8 * s, pol_stream);
                    tma_load_3d(kst_addr + s * kStageBytes + kStageBytes / 2, &tmK, 64, row, a.u0 + u, bar_kfull + 8 * s, pol_stream);
                    issued = T + 1;
                }
                w.advance(x);
            }
            if (!ok) {   // give up: let the copies already in flight land before the CTA exits
                int dummy = 0;
                for (int T = max(0, issued - SK); T < issued; ++T)
                    mbar_wait(bar_kfull + 8 * (T % SK), (uint32_t)((T / SK) & 1), &dummy, kWaitDrain, kWaitCycles);
                if (rings > 0) mbar_wait(bar_qfull, (uint32_t)((rings - 1) & 1), &dummy, kWaitDrain, kWaitCycles);
            }
        }
        // lanes 1-31 skipped the loop: the warp must be whole again before it reaches the CTA barrier of the tail
        // (bar.sync is an aligned instruction; lanes of one warp arriving at different times is undefined)
        __syncwarp();
    } else if (warp == 2) {
        // ------------------------------------------------ TMA producer: V tiles (one lane)
        if (lane == 0) {
            Walk w(a.U * NCe, n, (int)gridDim.x, (int)blockIdx.x);
            Item x;
            int issued = 0;                                 // V tiles loaded so far (only main chunks read V)
            bool ok = true;
            RingPos rv(0, SV);
            const uint64_t pol_stream = l2_policy_evict_first();
            while (ok && w.next(x)) {
                const int u = MC ? x.unit / NCe : x.unit;
                const bool main_item = MC ? (NCe == 1 || x.unit - u * NCe == c_main) : true;
                for (int j = 0; main_item && j < x.nk && ok; ++j, rv.step(1, SV)) {
                    const int s = rv.idx;
                    ok = mbar_wait(bar_vempty + 8 * s, (uint32_t)(rv.lap ^ 1), abort_flag, kWaitVEmpty, WL);
                    if (!ok) break;
                    const int row = (x.tile0 + j) * kTile;
                    mbar_expect_tx(bar_vfull + 8 * s, kStageBytes);
                    tma_load_3d(vst_addr + s * kStageBytes, &tmV, 0, row, a.u0 + u, bar_vfull + 8 * s, pol_stream);
                    tma_load_3d(vst_addr + s * kStageBytes + kStageBytes / 2, &tmV, 64, row, a.u0 + u, bar_vfull + 8 * s, pol_stream);
                    ++issued;
                }
                w.advance(x);
            }
            if (!ok) {
                int dummy = 0;
                for (int T = max(0, issued - SV); T < issued; ++T)
                    mbar_wait(bar_vfull + 8 * (T % SV), (uint32_t)((T / SV) & 1), &dummy, kWaitDrain, kWaitCycles);
            }
        }
        __syncwarp();       // see the K producer
    } else if (warp == 1) {
        // ------------------------------------------------ new-query substitution + MMA issue
        Walk w(a.U * NCe, n, (int)gridDim.x, (int)blockIdx.x);
        Item x;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(RGP >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
        bool ok = true;
        int n_mma = 0;                                  // tiles whose MMAs have been issued and committed
        RingPos rk(0, SK), rb(0, NB);
        while (ok && w.next(x)) {
            {
                if (w.nitems > 0 && lane == 0) umma_commit(bar_qempty);   // MMAs of the previous unit done with the ring
                // the new query replaces ring row t % R (the row of the token leaving the window)
                const int u = MC ? x.unit / NCe : x.unit;
                const bool main_item = MC ? (NCe == 1 || x.unit - u * NCe == c_main) : true;   // the chunk with the new query's slot
                uint4 qv[kMaxGroup / 2];
                const uint4 *qsrc = reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(a.q) + (size_t)u * a.Gq * kD);
#pragma unroll
                for (int i = 0; i < (G * 16 + 31) / 32; ++i)
                    if (lane + 32 * i < G * 16) qv[i] = lane + 32 * i < a.Gq * 16 ? qsrc[lane + 32 * i] : make_uint4(0, 0, 0, 0);
                ok = __all_sync(0xffffffffu, mbar_wait(bar_qfull, (uint32_t)(w.nitems & 1), abort_flag, kWaitQFull, WL));
                if (!ok) break;
#pragma unroll
                for (int i = 0; i < (G * 16 + 31) / 32; ++i) {
                    const int c = lane + 32 * i;
                    if (c < G * 16 && main_item) {
                        const int row = rs_loc * G + c / 16, ch = c % 16;
                        const uint32_t off = (uint32_t)((ch >> 3) * (RGP * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4));
                        *reinterpret_cast<uint4 *>(smem + L.q + off) = qv[i];
                    }
                }
                fence_proxy_async();
                __syncwarp();
            }
            for (int j = 0; j < x.nk; ++j, rk.step(1, SK), rb.step(1, NB)) {
                const int s = rk.idx, b = rb.idx;
                bool k = mbar_wait(bar_kfull + 8 * s, (uint32_t)rk.lap, abort_flag, kWaitKFull, WL);
                k = k && mbar_wait(bar_tempty + 8 * b, (uint32_t)(rb.lap ^ 1), abort_flag, kWaitTEmpty, WL);
                ok = __all_sync(0xffffffffu, k);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t d_tmem = tmem_base + (uint32_t)(b * RGP);
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint64_t ad = smem_desc_sw128(kst_addr + s * kStageBytes + (ks >> 2) * (kStageBytes / 2) + (ks & 3) * 32);
                        const uint64_t bd = smem_desc_sw128(q_addr + (ks >> 2) * (RGP * 128) + (ks & 3) * 32);
                        umma_bf16(d_tmem, ad, bd, idesc, ks > 0 ? 1u : 0u);
                    }
                    umma_commit(bar_kempty + 8 * s);      // K tile consumed
                    umma_commit(bar_tfull + 8 * b);       // accumulators ready
                }
                ++n_mma;
                __syncwarp();
            }
            w.advance(x);
        }
        // A tcgen05.commit arrives on its mbarrier asynchronously, when the MMAs before it have completed.  The
        // arrivals on the K-empty barriers of the last tiles have no waiter left (the producer has issued its last
        // load), and after a wait has given up the accumulator-full arrivals may have none either.  This warp
        // observes every one of them before the CTA frees its TMEM and exits, so that no MMA is still running and
        // no arrival can land in shared memory that by then belongs to a CTA of the next launch.
        {
            int dummy = 0;
            for (int T = max(0, n_mma - SK); T < n_mma; ++T)
                mbar_wait(bar_kempty + 8 * (T % SK), (uint32_t)((T / SK) & 1), &dummy, kWaitDrain, kWaitCycles);
            if (!ok)
                for (int T = max(0, n_mma - NB); T < n_mma; ++T)
                    mbar_wait(bar_tfull + 8 * (T % NB), (uint32_t)((T / NB) & 1), &dummy, kWaitDrain, kWaitCycles);
            __syncwarp();
        }
    } else if (warp < kFirstComputeWarp + 4 * NG) {
        // ------------------------------------------------ compute warps
        const int cw = warp - kFirstComputeWarp;     // 0 .. 4*NG-1
        const int grp = cw >> 2;                     // tile T belongs to group T % NG
        const int wq = warp & 3;                     // TMEM lane quarter of this warp
        const int gtid = wq * 32 + lane;             // position among the group's 128 key lanes
        float *wbuf = reinterpret_cast<float *>(smem + L.wbuf) + cw * G * kD;            // [g][d]
        float *wml = reinterpret_cast<float *>(smem + L.wml) + cw * 2 * kMaxGroup;         // [g][2]
        float *negc = reinterpret_cast<float *>(smem + L.negc) + cw * RGP;
        float *st_w = reinterpret_cast<float *>(smem + L.stw) + cw * (G * 32 + 2 * kMaxGroup);   // [g][lane]
        float *fac = st_w + G * 32, *mref = fac + kMaxGroup;         // warp-private, indexed by head
        const int RG = a.R * G;
        const int gid = lane >> 2, tig = lane & 3;
        constexpr int NT = G > 8 ? 2 : 1;            // 8-head column tiles of the transposed output

        // Running soft-max state of this warp over its keys of the open unit: reference max
        // per head (replicated in every lane), this lane's share of the denominator and of the
        // un-normalised output O^T[d][g].
        float mrun[G];
        float acc[NT][8][4];
        float lsum[NT];
        int seg_tiles = 0;
        int npub = 0;                                  // partials this warp has handed to the epilogue group

        Walk w(a.U * NCe, n, (int)gridDim.x, (int)blockIdx.x);
        Item x;
        bool ok = true;
        int Tn = grp;                                  // next tile of this group
        int skipped = 0;                               // MC: tiles of the items that read no V
        RingPos rb(grp, NB), rv(grp, SV);
        while (w.next(x)) {
            const int u = MC ? x.unit / NCe : x.unit;
            const int cc = MC ? (NCe == 1 ? c_main : x.unit - u * NCe) : 0;      // ring chunk of this item
            const bool main_item = MC ? cc == c_main : true;
            const UnitStep us = RAGGED ? unit_step(a, u, t, n, steps_done, evict) : UnitStep{n, 0, evict};   // the unit's own fill and policy decision
            {
                // frozen normalisers of the ring rows, negated; the new row and padding give weight 0
                for (int c = lane; c < RGP; c += 32) {
                    float v = -INFINITY;
                    const int row = MC ? cc * RGP + c : c;
                    if (row < RG && row / G != rs_new) v = -a.ring_c[(size_t)u * RG + row];
                    negc[c] = v;
                }
#pragma unroll
                for (int g = 0; g < G; ++g) mrun[g] = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    lsum[nt] = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) { acc[nt][i][0] = 0.f; acc[nt][i][1] = 0.f; acc[nt][i][2] = 0.f; acc[nt][i][3] = 0.f; }
                }
                seg_tiles = 0;
                __syncwarp();
            }
            float *s_new = a.s_new + (size_t)u * G * a.cap;
            float *Fdst = MC ? a.Fc + ((size_t)u * geo.nc + cc) * a.cap : a.F + (size_t)u * a.cap;
            if constexpr (MC) {
                if (main_item) {
                    rv = RingPos(Tn - skipped, SV);      // V tiles are numbered over the main items only
                } else {
                    // a chunk without the new query: fused scores of its rows over this group's tiles, nothing else
                    for (; Tn < w.T0 + x.nk && ok; Tn += NG, rb.step(NG, NB)) {
                        const int buf = rb.idx;
                        ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, (uint32_t)rb.lap, abort_flag, kWaitTFull, WL));
                        if (!ok) break;
                        tc_fence_after();
                        const int key = (x.tile0 + (Tn - w.T0)) * kTile + gtid;
                        const uint32_t taddr = tmem_base + (uint32_t)(buf * RGP) + ((uint32_t)(wq * 32) << 16);
                        float F = 0.f;
                        for (int c = 0; c < RGP; c += 32) {
                            uint32_t v[32];
                            tmem_ld32(taddr + (uint32_t)c, v);
                            score_chunk<G, FUSION>(v, negc + c, a.scale2, F);
                        }
                        if (key < us.n) Fdst[key] = F;
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                    }
                    skipped += x.nk;
                }
            }
            // this group's tiles are T = grp, grp + NG, ...: walk them directly
            for (; main_item && Tn < w.T0 + x.nk && ok; Tn += NG, rb.step(NG, NB), rv.step(NG, SV)) {
                const int j = Tn - w.T0;
                const int buf = rb.idx;
                // ---- scores of this warp's 32 keys (Eq. 4-6) and the new row's logits
                ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, (uint32_t)rb.lap, abort_flag, kWaitTFull, WL));
                if (!ok) break;
                tc_fence_after();
                const int key = (x.tile0 + j) * kTile + gtid;
                const bool valid = key < us.n;
                const uint32_t taddr = tmem_base + (uint32_t)(buf * RGP) + ((uint32_t)(wq * 32) << 16);
                // Each TMEM load and its wait form one asm statement: the destination registers are
                // written asynchronously, so nothing may touch them between the two.
                uint32_t sv[G];
                tmem_ld_n<G>(taddr + (uint32_t)(rs_loc * G), sv);

                // ---- online soft-max of the new row over this warp's keys (Eq. 1)
                bool changed = false;
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float s2 = valid ? __uint_as_float(sv[g]) * a.scale2 : -INFINITY;
                    st_w[g * 32 + lane] = s2;
                    if (valid && (us.evict || stored)) s_new[(size_t)g * a.cap + key] = s2;
                    const float mn = fmaxf(mrun[g], warp_max(s2));
                    // factor that brings what was accumulated under the old reference to the new one
                    const float f = mn == mrun[g] ? 1.f : ex2f(mrun[g] - mn);
                    changed |= mn != mrun[g];
                    mrun[g] = mn;
                    if (lane == 0) { fac[g] = f; mref[g] = mn == -INFINITY ? 0.f : mn; }
                }
                __syncwarp();
                if (changed && seg_tiles > 0) {
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int gr = gid + 8 * nt, gc = tig * 2 + 8 * nt;
                        const float fr = gr < G ? fac[gr] : 0.f, f0 = gc < G ? fac[gc] : 0.f, f1 = gc + 1 < G ? fac[gc + 1] : 0.f;
                        lsum[nt] *= fr;
#pragma unroll
                        for (int i = 0; i < 8; ++i) { acc[nt][i][0] *= f0; acc[nt][i][1] *= f1; acc[nt][i][2] *= f0; acc[nt][i][3] *= f1; }
                    }
                }

                // ---- O^T[d][g] += V^T[d][keys] . P^T[keys][g] over this warp's 32 keys.  This runs before the scoring
                // of the ring rows so that the V stage goes back to its producer as early as possible.
                const int s = rv.idx;
                // A V stage serves the two compute groups in turn whenever the ring has an odd number of stages, and
                // a parity wait cannot tell "this load has landed" from "the load before the previous one has
                // landed".  The accumulator buffers keep the groups close enough for that never to matter; waiting
                // for the previous load of the stage to be consumed first (the wait the producer does before it
                // refills the stage) makes the full barrier's parity unambiguous without relying on that.
                bool vok = mbar_wait(bar_vempty + 8 * s, (uint32_t)(rv.lap ^ 1), abort_flag, kWaitVEmpty, WL);
                vok = vok && mbar_wait(bar_vfull + 8 * s, (uint32_t)rv.lap, abort_flag, kWaitVFull, WL);
                ok = __all_sync(0xffffffffu, vok);
                if (!ok) break;
                const uint32_t vbase = vst_addr + s * kStageBytes;
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    uint32_t bhi[NT][2], blo[NT][2];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        // branch-free on purpose: ldmatrix / mma.sync below are .aligned and need the
                        // whole warp converged; lanes whose row is not a head compute and discard
                        const int gr = gid + 8 * nt;
                        const bool live = gr < G;
                        const int grc = live ? gr : 0;
                        const float *sp = st_w + grc * 32 + ks * 16 + tig * 2;
                        const float2 sa = *reinterpret_cast<const float2 *>(sp), sb = *reinterpret_cast<const float2 *>(sp + 8);
                        const float m = mref[grc];
                        float p0 = ex2f(sa.x - m), p1 = ex2f(sa.y - m), p2 = ex2f(sb.x - m), p3 = ex2f(sb.y - m);
                        p0 = live ? p0 : 0.f; p1 = live ? p1 : 0.f; p2 = live ? p2 : 0.f; p3 = live ? p3 : 0.f;
                        lsum[nt] += (p0 + p1) + (p2 + p3);
                        split_bf16x2(p0, p1, bhi[nt][0], blo[nt][0]);
                        split_bf16x2(p2, p3, bhi[nt][1], blo[nt][1]);
                    }
                    __syncwarp();
                    const int mat = lane >> 3, r = lane & 7;
                    const int krow = wq * 32 + ks * 16 + (mat >> 1) * 8 + r;
#pragma unroll
                    for (int db = 0; db < 8; ++db) {
                        const int ch = db * 2 + (mat & 1);
                        const uint32_t addr = vbase + (uint32_t)((ch >> 3) * (kStageBytes / 2) + krow * 128 + (((ch & 7) ^ (krow & 7)) << 4));
                        uint32_t af[4];
                        ldmatrix_x4_trans(addr, af);      // V^T fragment: rows = 16 d, columns = 16 keys
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            mma_bf16_16816(acc[nt][db], af, bhi[nt][0], bhi[nt][1]);
                            mma_bf16_16816(acc[nt][db], af, blo[nt][0], blo[nt][1]);
                        }
                    }
                }
                // The V tile was read through the generic proxy (ldmatrix); the producer refills the stage through the
                // async proxy (TMA).  An mbarrier arrive/wait pair orders accesses of one proxy only, so every lane
                // fences its reads against later async-proxy writes before the stage is handed back.  Without this
                // fence a refill now and then overtook the last reads of a tile (one 16-column block of one warp's
                // keys came out wrong, about ten times in 48 steps of 256 units).
                fence_proxy_async();
                __syncwarp();                               // every lane has read its rows of the V tile
                if (lane == 0) mbar_arrive(bar_vempty + 8 * s);
                __syncwarp();                               // converged again in front of the .aligned TMEM loads

                // ---- fused scores of this warp's 32 keys over the ring rows (Eq. 4-6): only on steps that run the
                // policy.  While the cache is still filling, and between two runs of a coarse-grained policy, nothing
                // is evicted and the accumulator buffer goes back as soon as the new row's logits have been read.
                if (us.evict && !stored) {
                    float F = 0.f;
                    for (int c = 0; c < RGP; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(taddr + (uint32_t)c, v);
                        score_chunk<G, FUSION>(v, negc + c, a.scale2, F);
                    }
                    if (valid) Fdst[key] = F;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                ++seg_tiles;
            }


            // ---- the item is done: leave this warp's partial for the epilogue group
            if (ok) {
                // the previous partial must have been read before its buffer is overwritten
                if (npub > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_pfree + 8 * cw, (uint32_t)((npub - 1) & 1), abort_flag, kWaitPFree, WL));
                if (ok) {
#pragma unroll
                    for (int nt = 0; nt < NT && main_item; ++nt) {
                        const int gr = gid + 8 * nt, gc = tig * 2 + 8 * nt;
                        float l = lsum[nt];
                        l += __shfl_xor_sync(0xffffffffu, l, 1);
                        l += __shfl_xor_sync(0xffffffffu, l, 2);
                        float m = -INFINITY;
#pragma unroll
                        for (int g = 0; g < G; ++g) m = g == gr ? mrun[g] : m;
                        if (tig == 0 && gr < G) { wml[gr * 2] = m; wml[gr * 2 + 1] = l; }
#pragma unroll
                        for (int db = 0; db < 8; ++db) {
                            if (gc < G) { wbuf[gc * kD + db * 16 + gid] = acc[nt][db][0]; wbuf[gc * kD + db * 16 + gid + 8] = acc[nt][db][2]; }
                            if (gc + 1 < G) { wbuf[(gc + 1) * kD + db * 16 + gid] = acc[nt][db][1]; wbuf[(gc + 1) * kD + db * 16 + gid + 8] = acc[nt][db][3]; }
                        }
                    }
                    // Fused scores / new-row logits of this warp's keys are read by the epilogue group of this CTA,
                    // or of another CTA when the unit is shared.  The arrive releases this warp's writes at CTA
                    // scope; for a shared unit the epilogue thread that takes the unit's ticket fences at device
                    // scope after it has observed the arrivals, which carries these writes along (release
                    // sequences are cumulative), so no device-scope fence is paid here.
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_udone);
                    ++npub;
                }
            }
            w.advance(x);
        }
    } else {
        // ------------------------------------------------ epilogue group (128 threads)
        const int etid = tid - (kFirstComputeWarp + 4 * NG) * 32;
        constexpr int NCW = 4 * NG;
        constexpr int kEpiBar = 1;
        const float *wbuf = reinterpret_cast<const float *>(smem + L.wbuf);
        const float *wml = reinterpret_cast<const float *>(smem + L.wml);
        float *epi = reinterpret_cast<float *>(smem + L.epi);
        float *fin_sm = epi;                                          // kFinFloats
        int *flag = reinterpret_cast<int *>(epi + kFinFloats);
        float *cml = epi + kFinFloats + 8;                            // merged (m, l) [g][2]
        float *sc = cml + 2 * kMaxGroup;                              // [warp][g] scale to the merged reference
        Walk w(a.U * NCe, n, (int)gridDim.x, (int)blockIdx.x);
        Item x;
        bool ok = true;
        int k = 0;                                                    // units finished so far
        while (ok && w.next(x)) {
            {
                const int u = MC ? x.unit / NCe : x.unit;
                const bool main_item = MC ? (NCe == 1 || x.unit - u * NCe == c_main) : true;
                const UnitStep us = RAGGED ? unit_step(a, u, t, n, steps_done, evict) : UnitStep{n, 0, evict};
                if (group_any(kEpiBar, !mbar_wait(bar_udone, (uint32_t)(k & 1), abort_flag, kWaitUDone, WL))) { ok = false; break; }
                // merge the compute warps' partials: common reference = max of theirs
                if (etid < G && main_item) {
                    float m = -INFINITY;
                    for (int cwi = 0; cwi < NCW; ++cwi) m = fmaxf(m, wml[cwi * 2 * kMaxGroup + etid * 2]);
                    float l = 0.f;
                    for (int cwi = 0; cwi < NCW; ++cwi) {
                        const float mw = wml[cwi * 2 * kMaxGroup + etid * 2];
                        const float f = mw == -INFINITY ? 0.f : ex2f(mw - m);
                        sc[cwi * kMaxGroup + etid] = f;
                        l += wml[cwi * 2 * kMaxGroup + etid * 2 + 1] * f;
                    }
                    cml[etid * 2] = m;
                    cml[etid * 2 + 1] = l;
                }
                group_sync(kEpiBar, kGroupThreads);
                float o[G];
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float v = 0.f;
#pragma unroll
                    for (int cwi = 0; cwi < NCW; ++cwi) v += wbuf[(cwi * G + g) * kD + etid] * sc[cwi * kMaxGroup + g];
                    o[g] = v;
                }
                group_sync(kEpiBar, kGroupThreads);                       // every warp buffer has been read
                if (etid < NCW) mbar_arrive(bar_pfree + 8 * etid);
                int my_index;
                const int ncta = w.ctas_of_unit(x.unit, my_index);
                if constexpr (MC) {
                    // Every (CTA, chunk) item of a unit takes one ticket; the items of the main chunk publish their
                    // partial of the attention output first.  The last item of the unit combines the chunks' fused
                    // scores and finishes the unit with the general epilogue.
                    if (main_item) {
                        float *pml = a.part_ml + ((size_t)u * a.splits + my_index) * G * 2;
                        float *po = a.part_o + ((size_t)u * a.splits + my_index) * G * kD;
#pragma unroll
                        for (int g = 0; g < G; ++g) po[g * kD + etid] = o[g];
                        if (etid < 2 * G) pml[etid] = cml[etid];
                    }
                    group_sync(kEpiBar, kGroupThreads);
                    if (etid == 0) {
                        int items = 0, idx;
                        for (int c = 0; c < NCe; ++c) items += w.ctas_of_unit(u * NCe + c, idx);
                        __threadfence();
                        const int last = atomicAdd(&a.ticket[u], 1) == items - 1;
                        __threadfence();
                        *flag = last;
                    }
                    group_sync(kEpiBar, kGroupThreads);
                    if (*flag) {
                        if (us.evict && !stored) {
                            float *F = a.F + (size_t)u * a.cap;
                            const float *Fc = a.Fc + (size_t)u * geo.nc * a.cap;
                            for (int key = etid; key < us.n; key += kGroupThreads) {
                                float f = __ldcg(Fc + key);
                                for (int c = 1; c < NCe; ++c) f = fuse(FUSION, f, __ldcg(Fc + (size_t)c * a.cap + key));
                                F[key] = f;
                            }
                            group_sync(kEpiBar, kGroupThreads);
                        }
                        int idx;
                        const int ncta_main = w.ctas_of_unit(u * NCe + (NCe == 1 ? 0 : c_main), idx);
                        finalize_unit<__nv_bfloat16, kD, G, true>(a, u, t, us.n, ncta_main, us.evict, fin_sm, etid, kGroupThreads,
                                                                  kEpiBar, RAGGED ? us.shift : 0);
                    }
                } else if (ncta == 1) {
                    finalize_fast<G, true>(a, u, t, us.n, 1, us.evict, fin_sm, etid, kEpiBar, o, cml, RAGGED ? us.shift : 0);
                } else {
                    // the unit is shared: publish this CTA's partial; the last CTA to do so finishes the unit.
                    // The group barrier orders every thread's writes (and, through the mbarrier above, the compute
                    // warps' writes) before the ticket thread's device-scope fence, which releases them all; the
                    // fence after the ticket is the acquire side, and the data is then read past L1 (ld.global.cg).
                    float *pml = a.part_ml + ((size_t)u * a.splits + my_index) * G * 2;
                    float *po = a.part_o + ((size_t)u * a.splits + my_index) * G * kD;
#pragma unroll
                    for (int g = 0; g < G; ++g) po[g * kD + etid] = o[g];
                    if (etid < 2 * G) pml[etid] = cml[etid];
                    group_sync(kEpiBar, kGroupThreads);
                    if (etid == 0) {
                        // release: the group's writes above (ordered before this thread by the barrier) become visible
                        // to whoever observes the ticket; acquire: the last arriver's reads below see the others'
                        int old;
                        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(a.ticket + u) : "memory");
                        *flag = old == ncta - 1;
                    }
                    group_sync(kEpiBar, kGroupThreads);
                    if (*flag) {
                        if (ncta <= 8 && ncta * G * 2 <= 256)
                            finalize_fast<G, false>(a, u, t, us.n, ncta, us.evict, fin_sm, etid, kEpiBar, o, nullptr, RAGGED ? us.shift : 0);
                        else
                            finalize_unit<__nv_bfloat16, kD, G>(a, u, t, us.n, ncta, us.evict, fin_sm, etid, kGroupThreads, kEpiBar,
                                                                RAGGED ? us.shift : 0);
                    }
                }
                group_sync(kEpiBar, kGroupThreads);
                ++k;
            }
            w.advance(x);
        }
    }

    // ------------------------------------------------ tail
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)geo.tmem_cols);
    }
    if (tid == 0 && *abort_flag) atomicCAS(&a.st->err, 0, *abort_flag);      // the first wait that gave up
}

}  // namespace

struct TcPlan {
    CUtensorMap tmK, tmV, tmQ;
    TcGeom geo;
    bool attr_set[5][2][3];
};

namespace {

int group_index(int G) { return G == 1 ? 0 : G == 2 ? 1 : G == 4 ? 2 : G == 8 ? 3 : G == 16 ? 4 : -1; }

template <int G, int FUSION, int NG, bool MC, bool RAGGED>
cudaError_t launch_gfn(TcPlan *plan, const DecodeArgs &a, cudaStream_t stream)
{
    auto kern = decode_tc_kernel<G, FUSION, NG, MC, RAGGED>;
    bool &set = plan->attr_set[group_index(G)][FUSION][MC ? 1 : RAGGED ? 2 : 0];
    if (!set) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan->geo.smem_bytes);
        if (e != cudaSuccess) return e;
        set = true;
    }
    // launched with programmatic stream serialisation: the kernel orders itself behind its predecessor with
    // griddepcontrol.wait (see the kernel's prologue)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan->geo.grid);
    cfg.blockDim = dim3(tc_threads(NG));
    cfg.dynamicSmemBytes = plan->geo.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a, plan->tmK, plan->tmV, plan->tmQ, plan->geo);
}

template <int G, int FUSION>
cudaError_t launch_gf(TcPlan *plan, const DecodeArgs &a, cudaStream_t stream)
{
    if (plan->geo.nc > 1 || a.prof)
        return a.row_n ? cudaErrorInvalidValue : launch_gfn<G, FUSION, kComputeGroups, true, false>(plan, a, stream);
    return a.row_n ? launch_gfn<G, FUSION, kComputeGroups, false, true>(plan, a, stream)
                   : launch_gfn<G, FUSION, kComputeGroups, false, false>(plan, a, stream);
}

template <int G>
cudaError_t launch_g(TcPlan *plan, const DecodeArgs &a, cudaStream_t stream)
{
    return a.fusion == kFusionSum ? launch_gf<G, kFusionSum>(plan, a, stream) : launch_gf<G, kFusionMax>(plan, a, stream);
}

int pad32(int x) { return (x + 31) & ~31; }

}  // namespace

int tc_padded_group(int G)
{
    int g = 1;
    while (g < G) g *= 2;
    return g;
}

// Chunks the recent-query ring is cut into: one MMA takes at most 256 ring rows (N of the instruction, and with
// two accumulator buffers the 512 TMEM columns).
int tc_ring_chunks(int G, int R)
{
    const int rows = R * tc_padded_group(G);
    return rows <= 256 ? 1 : (rows + 255) / 256;
}

namespace {
constexpr int kMaxRingChunks = 8;
// rows of one chunk: the chunks are made equally wide (a multiple of 32, hence of the padded group)
int chunk_rows(int G, int R)
{
    const int rows = R * tc_padded_group(G), nc = tc_ring_chunks(G, R);
    return pad32((rows + nc - 1) / nc);
}
}  // namespace

// G: the model's GQA ratio; the kernel works with the group padded to a power of two
bool tc_shape_supported(bool f32, int D, int G, int R)
{
    if (f32 || D != kD || G < 1 || G > kMaxGroup || R < 1) return false;
    return tc_ring_chunks(G, R) <= kMaxRingChunks;
}

int tc_grid(int U, int cap, int splits_hint, int n_sm) { return sched_grid(U, cap, splits_hint, n_sm); }

int tc_partials_per_unit(int U, int cap, int grid) { return sched_partials_per_unit(U, cap, grid); }

cudaError_t tc_plan_create(TcPlan **out, const DecodeArgs &a, int grid, unsigned long long wait_limit_cycles, bool prefetch,
                           char *err, size_t err_len)
{
    *out = nullptr;
    TcPlan *p = new (std::nothrow) TcPlan;
    if (!p) return cudaErrorMemoryAllocation;
    memset(p, 0, sizeof(*p));
    int dev = 0, n_sm = 0, max_smem = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) { delete p; return e; }
    TcGeom &g = p->geo;
    const int G = a.G;
    g.nc = a.nc;
    g.rgpad = g.nc > 1 ? chunk_rows(a.Gq, a.R) : pad32(a.R * G);
    // stored-profile mode: nothing is scored, so the operand is the 32-row piece of the ring that holds the new
    // query's slot (the kernel's chunk arithmetic with 32-row chunks, of which only that one is ever walked)
    if (a.prof) g.rgpad = 32;
    if (!a.prof &&
        (g.nc != tc_ring_chunks(a.Gq, a.R) || g.rgpad > 256 || g.rgpad * g.nc < a.R * G || (g.nc > 1 && !a.Fc))) {
        snprintf(err, err_len, "tensor-core kernel: ring chunk geometry does not match the shape");
        delete p;
        return cudaErrorInvalidValue;
    }
    g.ng = kComputeGroups;
    g.nb = g.rgpad <= 128 ? 4 : 2;
    g.tmem_cols = 32;
    while (g.tmem_cols < g.nb * g.rgpad) g.tmem_cols *= 2;
    g.grid = grid;
    g.wait_cycles = wait_limit_cycles > 0 ? (long long)wait_limit_cycles : kWaitCycles;
    // Two tiles: what counts is that a CTA's first loads after the wait hit L2 (config 1: 56.1 instead of 57.1 us per
    // step with 1 to 3 tiles).  More is worse - 8 tiles cost 3 us, 32 tiles 10 us - because the prefetches compete
    // with the previous grid's last CTAs.  Prefetching the first item's query ring as well changed nothing.
    // A launch over one layer's few units, whose CTAs hold two tiles or so each, is slower with it (17.9 instead of
    // 16.9 us per call): the caller asks for it on the whole-stack plan only.
    g.prefetch_tiles = prefetch ? 2 : 0;
    // as many 32 KB stages as fit, split between the K ring (short-lived tiles) and the V ring
    int total_stages = 0;
    for (int st = 9; st >= 2; --st) {
        g.sk = 1; g.sv = st - 1;
        if (tc_smem_layout(g, G).total + 1024 <= max_smem) { total_stages = st; break; }
    }
    if (total_stages < 2) {
        snprintf(err, err_len, "tensor-core kernel: shared memory does not fit");
        delete p;
        return cudaErrorInvalidConfiguration;
    }
    g.sk = total_stages >= 7 ? 3 : total_stages >= 5 ? 2 : 1;
    if (g.nc > 1 && !a.prof && total_stages >= 4) g.sk = 2;      // most items of a chunked window read K only
    g.sv = total_stages - g.sk;
    g.smem_bytes = tc_smem_layout(g, G).total + 1024;
    if (!encode_map(&p->tmK, a.K, a.U, a.cap, kTile) || !encode_map(&p->tmV, a.V, a.U, a.cap, kTile) ||
        !encode_map(&p->tmQ, a.ring_q, a.U, a.R * G, g.rgpad)) {
        snprintf(err, err_len, "tensor-core kernel: cuTensorMapEncodeTiled failed");
        delete p;
        return cudaErrorInvalidValue;
    }
    *out = p;
    return cudaSuccess;
}

void tc_plan_destroy(TcPlan *plan) { delete plan; }

cudaError_t launch_decode_tc(TcPlan *plan, const DecodeArgs &a, cudaStream_t stream)
{
    switch (a.G) {
        case 1: return launch_g<1>(plan, a, stream);
        case 2: return launch_g<2>(plan, a, stream);
        case 4: return launch_g<4>(plan, a, stream);
        case 8: return launch_g<8>(plan, a, stream);
        case 16: return launch_g<16>(plan, a, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mkv
