// Prompt-phase scoring on the tensor cores (bf16, head_dim 128, GQA group in {1,2,4,8,16}; a window of more than 256
// rows R*G is scored in pieces of up to 256 rows, one pair of passes per piece, the pieces' scores fused in place).
//
// One application of Algorithm 1 to the whole prompt needs, for every older prompt token k, the fused score
// F[k] = sum_r / max_r of S_r[k], S_r[k] = sum over the GQA group of the causal soft-max weight window row r puts
// on k (Eq. 1, Eq. 4-6).  The weights need each row's soft-max normaliser over ALL prompt keys first, so the keys
// are read twice and nothing of size rows x P ever goes to global memory:
//   pass 1  logits[rows x keys] = Qwin . K_tile^T on tcgen05 with the window rows in the TMEM lanes: every thread
//           owns one row and keeps its running (max, sum) over the keys it may see (causal inside the window);
//           the key range of a unit can be split over CTAs, whose partial (max, sum) pairs are merged in pass 2.
//   pass 2  logits^T[keys x rows] = K_tile . Qwin^T with the keys in the lanes (the decode kernel's orientation):
//           every thread owns one key, turns its row of logits into weights exp2(s - c_row), sums them over the
//           group and fuses them over the window; F[k] is written for the candidates (P floats per unit).
// The selection (radix top-C on (F, position) keys), the gather of the kept rows and the ring set-up stay the
// kernels of mkv_prefill.cu.  CTA layout: warps 0-3 and 6-9 are two consumer groups (one TMEM lane quarter per
// warp); tiles alternate between the groups, so group g always reads accumulator buffer g and keeps its own
// running (max, sum) per row in pass 1.  Warp 4 feeds K tiles with TMA into a ring of 32 KB stages, warp 5 issues
// the MMAs into the two TMEM accumulator buffers.  Every wait is bounded; a wait that runs out raises an error
// word that the host reads after the call.
#include <stdio.h>

#include "mkv_common.cuh"
#include "mkv_kernels.h"
#include "mkv_sm100.cuh"

namespace mkv {

namespace {

constexpr int kPfMaxStages = 3;
constexpr int kPfThreads = 320;
constexpr int kPfGroups = 2;                 // consumer groups = accumulator buffers
enum PfWait { kPfKEmpty = 21, kPfKFull, kPfTEmpty, kPfTFull, kPfDrain };

struct PfArgs {
    const __nv_bfloat16 *qwin;   // [U][G][Rw][128]: the window queries of unit u are heads u*G .. u*G+G-1
    float *part_ml;              // [nb][splits * kPfGroups][qrows][2] pass-1 partial (max, sum) per window row, log2 domain
    float *ring_c;               // [U][R][G] arena: normaliser of the row of position p in ring slot p % R
    float *Fp;                   // [nb][P] fused scores of the batch's units
    int *err;                    // error word (0 = none)
    int ub0;                     // first unit of this batch
    int P, Rw, G, R;
    int Gq;                      // real heads per unit in qwin; heads Gq .. G-1 are padding
    int rows;                    // window rows of this launch; row = (window slot - i0) * G + head
    int i0;                      // first window slot of this launch (a wide window is scored piece by piece)
    int accumulate;              // pass 2: fuse the scores into Fp (a later piece) instead of writing them
    int qrows;                   // rows padded to a multiple of 128 (pass 1: MMA M blocks)
    int rpad;                    // rows padded to a multiple of 32 (pass 2: MMA N)
    int splits;                  // CTAs per unit along the keys
    int tmem_cols;
    int stages;                  // K stages: 2 with up to 128 window rows (two CTAs share an SM), else 3
    float scale2;
    long long wait_cycles;
};

__host__ __device__ inline int pf_stages(int qrows) { return qrows <= 128 ? 2 : kPfMaxStages; }
__host__ __device__ inline int pf_smem_bytes(int qrows) { return qrows * 256 + pf_stages(qrows) * kStageBytes + 2048 + 1024; }

template <int PASS, int G, int FUSION>
__global__ void __launch_bounds__(kPfThreads, 2)
prefill_tc_kernel(const __grid_constant__ PfArgs a, const __grid_constant__ CUtensorMap tmK)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = blockIdx.x, ul = blockIdx.y, u = a.ub0 + ul;
    const int QR = a.qrows, RB = QR / 128, kPfStages = a.stages;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t q_addr = sbase, kst_addr = sbase + QR * 256;
    float *negc = reinterpret_cast<float *>(smem + QR * 256 + kPfStages * kStageBytes);     // [256]
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + QR * 256 + kPfStages * kStageBytes + 1024);
    const uint32_t bar_kfull = smem_u32(bars), bar_kempty = smem_u32(bars + 4);
    const uint32_t bar_tfull = smem_u32(bars + 8), bar_tempty = smem_u32(bars + 10);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 12);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 13);
    const long long WL = a.wait_cycles;

    // key tiles of this CTA: pass 1 covers every prompt key, pass 2 the candidates (older than the window)
    const int nkeys = PASS == 1 ? a.P : a.P - a.Rw;
    const int nt = nkeys > 0 ? (nkeys + kTile - 1) / kTile : 0;
    const int per = (nt + a.splits - 1) / a.splits;
    const int t0 = sp * per, t1 = min(nt, t0 + per);
    const int ntile = max(0, t1 - t0);
    const int bufcols = PASS == 1 ? QR : a.rpad;

    if (tid == 0) {
        prefetch_tensormap(&tmK);
        for (int s = 0; s < kPfStages; ++s) { mbar_init(bar_kfull + 8 * s, 1); mbar_init(bar_kempty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 5) tmem_alloc(smem_u32(tmem_slot), (uint32_t)a.tmem_cols);
    // the window queries, K-major with the 128-byte swizzle the MMA descriptors expect: two 64-column panels of
    // QR rows; rows beyond the real ones are zero
    for (int c = tid; c < QR * 16; c += kPfThreads) {
        const int row = c >> 4, ch = c & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row < a.rows && row % G < a.Gq) {
            const int i = row / G, g = row % G;
            v = reinterpret_cast<const uint4 *>(a.qwin + (((size_t)u * a.Gq + g) * a.Rw + a.i0 + i) * kD)[ch];
        }
        const uint32_t off = (uint32_t)((ch >> 3) * (QR * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4));
        *reinterpret_cast<uint4 *>(smem + off) = v;
    }
    if (PASS == 2) {
        // merge the pass-1 partials of this unit's key splits into each row's normaliser c = max + log2(sum)
        for (int row = tid; row < 256; row += kPfThreads) {
            float nc = -INFINITY;                               // padding rows give weight 0
            if (row < a.rows) {
                const int np = a.splits * kPfGroups;
                const float *pm = a.part_ml + (size_t)ul * np * QR * 2;
                float m = -INFINITY;
                for (int s = 0; s < np; ++s) m = fmaxf(m, pm[((size_t)s * QR + row) * 2]);
                float l = 0.f;
                for (int s = 0; s < np; ++s) {
                    const float ms = pm[((size_t)s * QR + row) * 2];
                    if (ms > -INFINITY) l += pm[((size_t)s * QR + row) * 2 + 1] * exp2f(ms - m);
                }
                // a padding head (zero query) takes no part: normaliser +inf, weight 0
                const float c = row % G < a.Gq ? m + log2f(l) : INFINITY;
                nc = -c;
                if (sp == 0) {
                    const int i = row / G, g = row % G;
                    const int rslot = (a.P - a.Rw + a.i0 + i) % a.R;
                    a.ring_c[((size_t)u * a.R + rslot) * G + g] = c;
                }
            }
            negc[row] = nc;
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------ TMA producer of K tiles (one lane)
        if (lane == 0) {
            const uint64_t pol = l2_policy_evict_first();
            bool ok = true;
            int issued = 0;
            for (int j = 0; j < ntile && ok; ++j) {
                const int s = j % kPfStages;
                ok = mbar_wait(bar_kempty + 8 * s, (uint32_t)(((j / kPfStages) & 1) ^ 1), abort_flag, kPfKEmpty, WL);
                if (!ok) break;
                const int row = (t0 + j) * kTile;
                mbar_expect_tx(bar_kfull + 8 * s, kStageBytes);
                tma_load_3d(kst_addr + s * kStageBytes, &tmK, 0, row, u, bar_kfull + 8 * s, pol);
                tma_load_3d(kst_addr + s * kStageBytes + kStageBytes / 2, &tmK, 64, row, u, bar_kfull + 8 * s, pol);
                issued = j + 1;
            }
            if (!ok) {      // let the copies in flight land before the CTA exits
                int dummy = 0;
                for (int j = max(0, issued - kPfStages); j < issued; ++j)
                    mbar_wait(bar_kfull + 8 * (j % kPfStages), (uint32_t)((j / kPfStages) & 1), &dummy, kPfDrain, kWaitCycles);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ------------------------------------------------ MMA issue
        const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 4) << 24);   // M = 128
        bool ok = true;
        int n_mma = 0;
        for (int j = 0; j < ntile; ++j) {
            const int s = j % kPfStages, b = j & 1;
            bool k = mbar_wait(bar_kfull + 8 * s, (uint32_t)((j / kPfStages) & 1), abort_flag, kPfKFull, WL);
            k = k && mbar_wait(bar_tempty + 8 * b, (uint32_t)(((j >> 1) & 1) ^ 1), abort_flag, kPfTEmpty, WL);
            ok = __all_sync(0xffffffffu, k);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                if (PASS == 1) {
                    // rows in the lanes: D[128 rows x 128 keys] = Q_block . K_tile^T, one block of 128 rows at a time
                    const uint32_t idesc = idesc_base | ((uint32_t)(kTile >> 3) << 17);
                    for (int rb = 0; rb < RB; ++rb) {
                        const uint32_t d_tmem = tmem_base + (uint32_t)(b * bufcols + rb * 128);
#pragma unroll
                        for (int ks = 0; ks < kD / 16; ++ks) {
                            const uint64_t ad = smem_desc_sw128(q_addr + (ks >> 2) * (QR * 128) + rb * (128 * 128) + (ks & 3) * 32);
                            const uint64_t bd = smem_desc_sw128(kst_addr + s * kStageBytes + (ks >> 2) * (kStageBytes / 2) + (ks & 3) * 32);
                            umma_bf16(d_tmem, ad, bd, idesc, ks > 0 ? 1u : 0u);
                        }
                    }
                } else {
                    // keys in the lanes: D[128 keys x rpad rows] = K_tile . Q^T
                    const uint32_t idesc = idesc_base | ((uint32_t)(a.rpad >> 3) << 17);
                    const uint32_t d_tmem = tmem_base + (uint32_t)(b * bufcols);
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint64_t ad = smem_desc_sw128(kst_addr + s * kStageBytes + (ks >> 2) * (kStageBytes / 2) + (ks & 3) * 32);
                        const uint64_t bd = smem_desc_sw128(q_addr + (ks >> 2) * (QR * 128) + (ks & 3) * 32);
                        umma_bf16(d_tmem, ad, bd, idesc, ks > 0 ? 1u : 0u);
                    }
                }
                umma_commit(bar_kempty + 8 * s);
                umma_commit(bar_tfull + 8 * b);
            }
            ++n_mma;
            __syncwarp();
        }
        {   // every commit is observed before TMEM is freed and the CTA exits
            int dummy = 0;
            for (int j = max(0, n_mma - kPfStages); j < n_mma; ++j)
                mbar_wait(bar_kempty + 8 * (j % kPfStages), (uint32_t)((j / kPfStages) & 1), &dummy, kPfDrain, kWaitCycles);
            if (!ok)
                for (int j = max(0, n_mma - 2); j < n_mma; ++j)
                    mbar_wait(bar_tfull + 8 * (j & 1), (uint32_t)((j >> 1) & 1), &dummy, kPfDrain, kWaitCycles);
            __syncwarp();
        }
    } else {
        // ------------------------------------------------ consumers: one TMEM lane quarter per warp (a warp reads
        // the quarter warp % 4), group 0 = warps 0-3 takes the even tiles, group 1 = warps 6-9 the odd ones
        const int grp = warp < 4 ? 0 : 1;
        const int lq = (warp & 3) * 32 + lane;               // lane of the accumulator this thread reads
        const uint32_t tlane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        if (PASS == 1) {
            // this thread's rows (one per block of 128) and the last key each may see
            float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
            int lim[2];
#pragma unroll
            for (int rb = 0; rb < 2; ++rb) {
                const int row = rb * 128 + lq;
                lim[rb] = (rb < RB && row < a.rows) ? a.P - a.Rw + a.i0 + row / G : -1;
            }
            for (int j = grp; j < ntile && ok; j += kPfGroups) {
                const int b = grp;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * b, (uint32_t)((j >> 1) & 1), abort_flag, kPfTFull, WL));
                if (!ok) break;
                tc_fence_after();
                const int key0 = (t0 + j) * kTile;
#pragma unroll
                for (int rb = 0; rb < 2; ++rb) {
                    if (rb >= RB) break;
                    for (int c = 0; c < kTile; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(tlane + (uint32_t)(b * bufcols + rb * 128 + c), v);
                        const int kc = key0 + c;
                        if (kc <= lim[rb]) {                 // else: nothing this row may see in these 32 keys
                            if (kc + 31 > lim[rb]) {         // the row's causal limit falls inside the chunk
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (kc + i > lim[rb]) v[i] = 0xff800000u;        // -inf: weight 0
                            }
                            // the scale is positive, so the maximum is taken on the raw logits and scaled once;
                            // one FFMA per key then forms s * scale - m
                            float cm = -INFINITY;
#pragma unroll
                            for (int i = 0; i < 32; ++i) cm = fmaxf(cm, __uint_as_float(v[i]));
                            cm *= a.scale2;
                            if (cm > m[rb]) { l[rb] *= ex2f(m[rb] - cm); m[rb] = cm; }
                            const float nm = -m[rb];
                            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                acc0 += ex2f(fmaf(__uint_as_float(v[i]), a.scale2, nm));
                                acc1 += ex2f(fmaf(__uint_as_float(v[i + 1]), a.scale2, nm));
                            }
                            l[rb] += acc0 + acc1;
                        }
                        __syncwarp();                        // the lanes meet again in front of the aligned TMEM load
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * b);
                __syncwarp();
            }
            if (ok) {
                float *pm = a.part_ml + (((size_t)ul * a.splits + sp) * kPfGroups + grp) * QR * 2;
#pragma unroll
                for (int rb = 0; rb < 2; ++rb)
                    if (rb < RB) { pm[(rb * 128 + lq) * 2] = m[rb]; pm[(rb * 128 + lq) * 2 + 1] = l[rb]; }
            }
        } else {
            float *Fu = a.Fp + (size_t)ul * a.P;
            for (int j = grp; j < ntile && ok; j += kPfGroups) {
                const int b = grp;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * b, (uint32_t)((j >> 1) & 1), abort_flag, kPfTFull, WL));
                if (!ok) break;
                tc_fence_after();
                float F = 0.f;
                for (int c = 0; c < a.rpad; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(tlane + (uint32_t)(b * bufcols + c), v);
                    score_chunk<G, FUSION>(v, negc + c, a.scale2, F);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * b);
                __syncwarp();
                const int key = (t0 + j) * kTile + lq;
                if (key < nkeys) {
                    if (a.accumulate) F = FUSION == kFusionSum ? Fu[key] + F : fmaxf(Fu[key], F);   // Eq. 5 / 6 over the pieces
                    Fu[key] = F;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
    }
    if (tid == 0 && *abort_flag) atomicCAS(a.err, 0, *abort_flag);
}

template <int PASS, int G>
cudaError_t launch_pass(const PfArgs &a, const CUtensorMap &tm, int nb, int fusion, cudaStream_t stream)
{
    auto kern = fusion == kFusionSum ? prefill_tc_kernel<PASS, G, kFusionSum> : prefill_tc_kernel<PASS, G, kFusionMax>;
    const int smem = pf_smem_bytes(a.qrows);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    PfArgs b = a;
    const int cols = 2 * (PASS == 1 ? a.qrows : a.rpad);
    b.tmem_cols = 32;
    while (b.tmem_cols < cols) b.tmem_cols *= 2;
    kern<<<dim3(a.splits, nb), kPfThreads, smem, stream>>>(b, tm);
    return cudaGetLastError();
}

template <int PASS>
cudaError_t launch_pass_any(const PfArgs &a, const CUtensorMap &tm, int nb, int fusion, cudaStream_t stream)
{
    switch (a.G) {
        case 1: return launch_pass<PASS, 1>(a, tm, nb, fusion, stream);
        case 2: return launch_pass<PASS, 2>(a, tm, nb, fusion, stream);
        case 4: return launch_pass<PASS, 4>(a, tm, nb, fusion, stream);
        case 8: return launch_pass<PASS, 8>(a, tm, nb, fusion, stream);
        case 16: return launch_pass<PASS, 16>(a, tm, nb, fusion, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool prefill_tc_supported(bool f32, int D, int G, int R, const void *k, int P)
{
    // any window: the pieces need no more than 256 rows at a time (the decode kernel's own limit on the ring, which
    // the stored-profile mode lifts, does not apply here)
    return !f32 && D == kD && G >= 1 && G <= kMaxGroup && R >= 1 && ((uintptr_t)k & 15) == 0 && P >= 1;
}

int prefill_tc_splits(int units_in_batch, int P, int window_rows)
{
    // CTAs per unit along the keys.  A CTA pays a set-up (TMEM, barriers, the window queries into shared memory,
    // in pass 2 the merge of the partial normalisers) worth about `kSetupTiles` key tiles, and the grid runs in
    // waves of `slots` resident CTAs: take the split with the fewest tile-times over all waves.
    constexpr int kSetupTiles = 3;
    const int nt = (P + kTile - 1) / kTile;
    const int slots = 148 * (window_rows <= 128 ? 2 : 1);             // pieces of a wide window: one CTA per SM
    int best = 1;
    long long best_cost = -1;
    for (int s = 1; s <= nt && s <= 64; ++s) {
        const long long waves = ((long long)units_in_batch * s + slots - 1) / slots;
        const long long cost = waves * ((nt + s - 1) / s + kSetupTiles);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

size_t prefill_tc_floats_per_unit(int P, int Rw, int G, int splits)
{
    const int rows = Rw * G < 256 ? Rw * G : 256;                        // a launch scores at most 256 window rows
    const int qrows = ((rows + 127) / 128) * 128;
    return (size_t)P + (size_t)splits * kPfGroups * qrows * 2;
}

// Window-row normalisers into ring_c and fused scores of the prompt's older tokens into Fp [nb][P] for units
// ub0 .. ub0+nb-1.  `part` holds nb * splits * kPfGroups * qrows * 2 floats of scratch, `err` is a zeroed error word.
cudaError_t run_prefill_scores_tc(const DecodeArgs &a, const void *k, const void *qwin, int P, int ub0, int nb, int splits,
                                  float *Fp, float *part, int *err, unsigned long long *launches, cudaStream_t stream)
{
    CUtensorMap tm;
    if (!encode_map(&tm, const_cast<void *>(k), a.U, P, kTile)) return cudaErrorInvalidValue;
    PfArgs pa;
    pa.qwin = static_cast<const __nv_bfloat16 *>(qwin);
    pa.part_ml = part; pa.ring_c = a.ring_c; pa.Fp = Fp; pa.err = err;
    pa.ub0 = ub0; pa.P = P; pa.Rw = P < a.R ? P : a.R; pa.G = a.G; pa.R = a.R; pa.Gq = a.Gq;
    pa.splits = splits;
    pa.tmem_cols = 0;
    pa.scale2 = a.scale2;
    pa.wait_cycles = kWaitCycles;
    // up to 256 window rows per pair of passes; the rows of a wider window are taken in pieces of whole window
    // slots, whose normalisers are independent and whose scores fuse associatively (Eq. 5 / 6)
    const int slots_per_piece = 256 / a.G;
    for (int i0 = 0; i0 < pa.Rw; i0 += slots_per_piece) {
        pa.i0 = i0;
        pa.accumulate = i0 > 0 ? 1 : 0;
        pa.rows = min(slots_per_piece, pa.Rw - i0) * a.G;
        pa.qrows = ((pa.rows + 127) / 128) * 128;
        pa.rpad = (pa.rows + 31) & ~31;
        pa.stages = pf_stages(pa.qrows);
        cudaError_t e = launch_pass_any<1>(pa, tm, nb, a.fusion, stream);
        if (e != cudaSuccess) return e;
        e = launch_pass_any<2>(pa, tm, nb, a.fusion, stream);
        *launches += 2;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace mkv
