// Prompt phase of MorphKV (set-up, not part of the per-token hot path).
//
// The paper states no prefill procedure; this is one application of Algorithm 1 with the
// whole prompt as the cache G_i: the last Rw = min(R, P) prompt tokens are the window, each
// window row's attention profile is its causal soft-max over all prompt keys (Eq. 1), every
// older prompt token gets the fused score of Eq. 4-6 (group sum first), and the C best are
// kept beside the window (Eq. 7).  The selection is a block-wide radix select over
// (score, position) keys, so ties keep the lower position deterministically.
#include <mutex>

#include "mkv_common.cuh"
#include "mkv_kernels.h"

namespace mkv {

namespace {

constexpr int kPT = 256;    // threads per CTA
constexpr int kPK = 32;     // keys per tile
constexpr int kPR = 64;     // window rows per sub-block

__device__ __forceinline__ void ld4(const float *p, float (&o)[4])
{
    const float4 v = *reinterpret_cast<const float4 *>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
__device__ __forceinline__ void ld4(const __nv_bfloat16 *p, float (&o)[4])
{
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
}

__global__ void init_arena_kernel(DecodeArgs a)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t ncap = (size_t)a.U * a.cap;
    if (i < ncap) { a.pos[i] = -1; a.F[i] = 0.f; }
    if (i < (size_t)a.U * a.R * a.G) a.ring_c[i] = INFINITY;   // empty ring row: weight 0
    if (i < (size_t)a.U) { a.ticket[i] = 0; a.evicted_pos[i] = -1; }
}

// the whole-stack state and one state per layer (per-layer calls advance their own)
__global__ void set_state_kernel(DevState *st, int n_states, long long t, int n)
{
    for (int i = threadIdx.x; i < n_states; i += blockDim.x) {
        st[i].t = t; st[i].n = n; st[i].steps = 0; st[i].err = 0; st[i].done = 0; st[i].compact = 0;
    }
}

// S[ub][row = i*G + g][j] = log2-domain logit of window row (i, g) against prompt key j,
// -inf where j lies after the row's own position (causal mask).
template <typename T, int D>
__global__ void __launch_bounds__(kPT) prefill_logits_kernel(const T *__restrict__ k, const T *__restrict__ qwin,
                                                             float *__restrict__ S, int ub0, int P, int Rw, int G,
                                                             float scale2, int Ps, int Rws)
{
    // Ps, Rws: tokens per unit in k and entries per head in qwin as laid out by the caller (P and Rw unless the
    // batch rows' prompts have different lengths and the tensors are padded to the longest)
    extern __shared__ __align__(16) float psm[];
    float *Ks = psm, *Qs = psm + kPK * (D + 4), *Ssm = Qs + kPR * (D + 4);
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int u = ub0 + blockIdx.y, kt = blockIdx.x * kPK;
    const int rows = Rw * G;
    constexpr int KS = D + 4, C4 = D / 4;
    const T *Ku = k + (size_t)u * Ps * D;
    for (int idx = tid; idx < kPK * C4; idx += kPT) {
        const int key = idx / C4, c4 = idx % C4;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (kt + key < P) ld4(Ku + (size_t)(kt + key) * D + c4 * 4, v);
        *reinterpret_cast<float4 *>(Ks + key * KS + c4 * 4) = make_float4(v[0], v[1], v[2], v[3]);
    }
    for (int r0 = 0; r0 < rows; r0 += kPR) {
        const int nr = min(kPR, rows - r0);
        __syncthreads();
        for (int idx = tid; idx < nr * C4; idx += kPT) {
            const int rl = idx / C4, c4 = idx % C4;
            const int row = r0 + rl, i = row / G, g = row % G;
            float v[4];
            ld4(qwin + (((size_t)u * G + g) * Rws + i) * D + c4 * 4, v);
            *reinterpret_cast<float4 *>(Qs + rl * KS + c4 * 4) = make_float4(v[0], v[1], v[2], v[3]);
        }
        __syncthreads();
        float acc[2][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { acc[0][i] = 0.f; acc[1][i] = 0.f; }
        const float *ka = Ks + ty * KS, *kb = Ks + (ty + 16) * KS;
        const float *qr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) qr[i] = Qs + ((tx + 16 * i) < nr ? (tx + 16 * i) : 0) * KS;
#pragma unroll 4
        for (int dd = 0; dd < D; dd += 4) {
            const float4 x = *reinterpret_cast<const float4 *>(ka + dd);
            const float4 y = *reinterpret_cast<const float4 *>(kb + dd);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 qv = *reinterpret_cast<const float4 *>(qr[i] + dd);
                acc[0][i] += x.x * qv.x + x.y * qv.y + x.z * qv.z + x.w * qv.w;
                acc[1][i] += y.x * qv.x + y.y * qv.y + y.z * qv.z + y.w * qv.w;
            }
        }
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
            for (int i = 0; i < 4; ++i) Ssm[(ty + 16 * kk) * (kPR + 1) + tx + 16 * i] = acc[kk][i] * scale2;
        __syncthreads();
        for (int idx = tid; idx < nr * kPK; idx += kPT) {
            const int rl = idx / kPK, key = idx % kPK;
            const int j = kt + key;
            if (j >= P) continue;
            const int row = r0 + rl;
            const int rpos = P - Rw + row / G;           // absolute position of the window row
            S[((size_t)blockIdx.y * rows + row) * P + j] = (j <= rpos) ? Ssm[key * (kPR + 1) + rl] : -INFINITY;
        }
    }
}

// c = max + log2(sum exp2(s - max)) of one window row; stored in the ring row p % R.
__global__ void __launch_bounds__(kPT) prefill_rowstats_kernel(const float *__restrict__ S, float *__restrict__ ring_c,
                                                               int ub0, int P, int Rw, int G, int Gs, int R, int shift)
{
    __shared__ float red[kPT / 32];
    __shared__ float bc;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x, u = ub0 + blockIdx.y;
    const float *s = S + ((size_t)blockIdx.y * Rw * G + row) * P;
    float m = -INFINITY;
    for (int j = tid; j < P; j += kPT) m = fmaxf(m, s[j]);
    m = warp_max(m);
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (tid == 0) { float x = red[0]; for (int w = 1; w < kPT / 32; ++w) x = fmaxf(x, red[w]); bc = x; }
    __syncthreads();
    m = bc;
    float l = 0.f;
    for (int j = tid; j < P; j += kPT) l += exp2f(s[j] - m);
    l = warp_sum(l);
    __syncthreads();
    if (lane == 0) red[warp] = l;
    __syncthreads();
    if (tid == 0) {
        float x = 0.f;
        for (int w = 0; w < kPT / 32; ++w) x += red[w];
        const int i = row / G, g = row % G;
        const int rslot = (P - Rw + i + shift) % R;     // ring slots are assigned on the context's common time axis
        ring_c[((size_t)u * R + rslot) * Gs + g] = m + log2f(x);     // Gs: heads per ring slot (G padded)
    }
}

// Eq. 4-6 with Algorithm 1's group sum: F[j] for every older prompt token j < P - Rw.
__global__ void __launch_bounds__(kPT) prefill_fuse_kernel(const float *__restrict__ S, const float *__restrict__ ring_c,
                                                           float *__restrict__ Fp, int ub0, int P, int Rw, int G, int Gs,
                                                           int R, int fusion, int shift)
{
    extern __shared__ float cs[];   // [Rw * G]
    const int u = ub0 + blockIdx.y, rows = Rw * G;
    for (int row = threadIdx.x; row < rows; row += kPT) {
        const int rslot = (P - Rw + row / G + shift) % R;
        cs[row] = ring_c[((size_t)u * R + rslot) * Gs + row % G];
    }
    __syncthreads();
    const int j = blockIdx.x * kPT + threadIdx.x;
    if (j >= P - Rw) return;
    const float *s = S + (size_t)blockIdx.y * rows * P + j;
    float F = 0.f;
    for (int i = 0; i < Rw; ++i) {
        float Sr = 0.f;
        for (int g = 0; g < G; ++g) Sr += exp2f(s[(size_t)(i * G + g) * P] - cs[i * G + g]);
        F = fuse(fusion, F, Sr);
    }
    Fp[(size_t)blockIdx.y * P + j] = F;
}

// Top-C of the M = P - Rw older tokens by (F descending, position ascending): an 8-pass
// radix select finds the C-th best 64-bit rank key, then an order-preserving compaction
// lists the kept positions, followed by the window positions.
constexpr int kSelT = 1024;  // threads of the selection kernel: a pass is a chain of rounds of kSelT keys
__global__ void __launch_bounds__(kSelT) prefill_select_kernel(const float *__restrict__ Fp, int *__restrict__ pos, int ub0,
                                                               int P, int Rw, int C, int cap)
{
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long prefix_s;
    __shared__ int remaining_s, done_s;
    __shared__ int wtot[kSelT / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = ub0 + blockIdx.x, M = P - Rw;
    const float *F = Fp + (size_t)blockIdx.x * P;
    int *upos = pos + (size_t)u * cap;
    unsigned long long prefix = 0;
    int remaining = C;
    constexpr int kSelBatch = 4;                                         // keys per thread in flight
    for (int pass = 7; pass >= 0; --pass) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        const int shift = 8 * pass;
        for (int c0 = 0; c0 < M; c0 += kSelT * kSelBatch) {
            // the loads of a batch are issued together: a pass is a chain of L2 round trips otherwise
            unsigned int fb[kSelBatch];
#pragma unroll
            for (int i = 0; i < kSelBatch; ++i) {
                const int j = c0 + i * kSelT + tid;
                fb[i] = j < M ? __float_as_uint(F[j]) : 0u;
            }
#pragma unroll
            for (int i = 0; i < kSelBatch; ++i) {
                if (c0 + i * kSelT >= M) break;                          // uniform over the CTA
                const int j = c0 + i * kSelT + tid;
                unsigned int bin = 256u;                                 // 256: not counted in this pass
                if (j < M) {
                    const unsigned long long key = rank_key(fb[i], j);
                    if (pass == 7 || (key >> (shift + 8)) == prefix) bin = (unsigned)(key >> shift) & 255u;
                }
                // one shared-memory atomic per warp and distinct bucket: the high bytes of the keys (sign and
                // exponent of the score) fall into a few buckets, and 32 atomics on one word would be serialised
                const unsigned int peers = __match_any_sync(0xffffffffu, bin);
                if (bin < 256u && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], (unsigned)__popc(peers));
            }
        }
        __syncthreads();
        // the bucket b that holds the `remaining`-th best key: above(b) < remaining <= above(b) + hist[b], with
        // above(b) the number of keys in higher buckets.  Thread b < 256 owns bucket b; exactly one qualifies.
        int h = 0, incl = 0;
        if (tid < 256) {                                                 // whole warps 0..7
            h = (int)hist[tid];
            incl = h;                                                    // sum over this warp's buckets >= tid
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += up;
            }
            if (lane == 0) wtot[warp] = incl;
        }
        __syncthreads();
        if (tid < 256) {
            int above = incl - h;
            for (int w = warp + 1; w < 8; ++w) above += wtot[w];
            if (h > 0 && above < remaining && remaining <= above + h) {
                const unsigned long long np = (prefix << 8) | (unsigned long long)tid;
                // the bucket fills the remaining places exactly: every key in it is kept, so the smallest key with
                // this prefix is the threshold and the finer passes (mostly tie-breaking position bits) are not
                // needed
                const bool exact = above + h == remaining;
                remaining_s = remaining - above;
                prefix_s = exact ? np << shift : np;
                done_s = exact ? 1 : 0;
            }
        }
        __syncthreads();
        prefix = prefix_s;
        remaining = remaining_s;
        const bool done = done_s != 0;
        __syncthreads();
        if (done) break;
    }
    // order-preserving compaction of the kept positions, kSelT keys per round
    int base = 0;
    for (int c0 = 0; c0 < M; c0 += kSelT) {
        const int j = c0 + tid;
        const bool keep = j < M && rank_key(__float_as_uint(F[j]), j) >= prefix;
        const unsigned int bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) wtot[warp] = __popc(bal);
        __syncthreads();
        int incl = wtot[lane];                                           // every warp scans the 32 warp totals
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int dn = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += dn;
        }
        const int before = warp == 0 ? 0 : __shfl_sync(0xffffffffu, incl, warp - 1);
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (keep) upos[base + before + __popc(bal & ((1u << lane) - 1u))] = j;
        base += total;
        __syncthreads();
    }
    for (int i = tid; i < Rw; i += kSelT) upos[C + i] = M + i;
}

__global__ void prefill_identity_pos_kernel(int *pos, int U, int n, int cap)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)U * n) return;
    pos[(i / n) * cap + (i % n)] = (int)(i % n);
}

// K/V rows of the kept prompt positions into the arena, 16 bytes per thread.
template <typename T, int D>
__global__ void prefill_gather_kernel(const T *__restrict__ k, const T *__restrict__ v, DecodeArgs a, int Ps, int n)
{
    constexpr int CH = D * sizeof(T) / 16;
    const int u = blockIdx.x;
    const int idx = blockIdx.y * blockDim.x + threadIdx.x;
    if (idx >= n * CH) return;
    const int slot = idx / CH, c = idx % CH;
    const int p = a.pos[(size_t)u * a.cap + slot];
    const uint4 *ks = reinterpret_cast<const uint4 *>(k + ((size_t)u * Ps + p) * D) + c;
    const uint4 *vs = reinterpret_cast<const uint4 *>(v + ((size_t)u * Ps + p) * D) + c;
    reinterpret_cast<uint4 *>(static_cast<T *>(a.K) + ((size_t)u * a.cap + slot) * D)[c] = *ks;
    reinterpret_cast<uint4 *>(static_cast<T *>(a.V) + ((size_t)u * a.cap + slot) * D)[c] = *vs;
}

// window queries into their ring rows (row p % R)
template <typename T, int D>
__global__ void prefill_ring_kernel(const T *__restrict__ qwin, DecodeArgs a, int P, int Rw, int Rws, int shift)
{
    const int u = blockIdx.x, G = a.G, Gq = a.Gq;       // heads Gq .. G-1 of a ring slot are padding (zero query)
    T *rq = static_cast<T *>(a.ring_q) + (size_t)u * a.R * G * D;
    for (int idx = threadIdx.x; idx < Rw * G * D; idx += blockDim.x) {
        const int dd = idx % D, g = (idx / D) % G, i = idx / (D * G);
        const int rslot = (P - Rw + i + shift) % a.R;
        if (g < Gq) rq[((size_t)rslot * G + g) * D + dd] = qwin[(((size_t)u * Gq + g) * Rws + i) * D + dd];
        else stf(rq + ((size_t)rslot * G + g) * D + dd, 0.f);
    }
}

// the same, 16 bytes per thread (q_window 16-byte aligned)
template <typename T, int D>
__global__ void prefill_ring_vec_kernel(const T *__restrict__ qwin, DecodeArgs a, int P, int Rw, int Rws, int shift)
{
    constexpr int CH = D * sizeof(T) / 16;
    const int u = blockIdx.x, G = a.G, Gq = a.Gq;
    const int idx = blockIdx.y * blockDim.x + threadIdx.x;
    if (idx >= Rw * G * CH) return;
    const int c = idx % CH, g = (idx / CH) % G, i = idx / (CH * G);
    const int rslot = (P - Rw + i + shift) % a.R;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (g < Gq) v = reinterpret_cast<const uint4 *>(qwin + (((size_t)u * Gq + g) * Rws + i) * D)[c];
    reinterpret_cast<uint4 *>(static_cast<T *>(a.ring_q) + (((size_t)u * a.R + rslot) * G + g) * D)[c] = v;
}

// The prompt phase on a scratch area of `scratch_floats` floats (the window-row logits S and the fused scores of
// as many units as fit go through it, batch after batch).  Every element a kernel reads was written earlier in the
// same batch, so what the area held before never matters.
// CURRENT normalisation after the prompt-phase selection: each window row's normaliser is taken again over the
// tokens that were kept and that the row may see, c = log2 sum exp2(s), from the arena as it stands (kept K rows,
// their positions, the ring's queries).  One CTA per (window row, unit).
template <typename T, int D>
__global__ void __launch_bounds__(kPT) prefill_renorm_kernel(DecodeArgs a, int P, int Rw, int n, int shift)
{
    __shared__ float qs[D];
    __shared__ float red[kPT / 32];
    __shared__ float bc;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.y, G = a.G, row = blockIdx.x, i = row / G, g = row % G;
    const int rpos = P - Rw + i, rslot = (rpos + shift) % a.R;
    float *c_out = a.ring_c + ((size_t)u * a.R + rslot) * G + g;
    if (*c_out == INFINITY) return;                                   // padding head
    const T *q = static_cast<const T *>(a.ring_q) + (((size_t)u * a.R + rslot) * G + g) * D;
    for (int d = tid; d < D; d += kPT) qs[d] = ldf(q + d);
    __syncthreads();
    const T *K = static_cast<const T *>(a.K) + (size_t)u * a.cap * D;
    const int *pos = a.pos + (size_t)u * a.cap;
    float s[8];       // up to 8 slots per thread per round
    float m = -INFINITY, l = 0.f;
    for (int k0 = 0; k0 < n; k0 += 8 * kPT) {
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const int k = k0 + b * kPT + tid;
            s[b] = -INFINITY;
            if (k < n && pos[k] <= rpos) {
                float acc = 0.f;
                for (int d = 0; d < D; ++d) acc += qs[d] * ldf(K + (size_t)k * D + d);
                s[b] = acc * a.scale2;
            }
        }
        float cm = m;
#pragma unroll
        for (int b = 0; b < 8; ++b) cm = fmaxf(cm, s[b]);
        if (cm > m) { l *= exp2f(m - cm); m = cm; }
        if (m > -INFINITY)
#pragma unroll
            for (int b = 0; b < 8; ++b) l += exp2f(s[b] - m);
    }
    float bm = warp_max(m);
    if (lane == 0) red[warp] = bm;
    __syncthreads();
    if (tid == 0) { float x = red[0]; for (int w = 1; w < kPT / 32; ++w) x = fmaxf(x, red[w]); bc = x; }
    __syncthreads();
    bm = bc;
    float bl = warp_sum(m > -INFINITY ? l * exp2f(m - bm) : 0.f);
    __syncthreads();
    if (lane == 0) red[warp] = bl;
    __syncthreads();
    if (tid == 0) {
        float x = 0.f;
        for (int w = 0; w < kPT / 32; ++w) x += red[w];
        *c_out = bm + log2f(x);
    }
}

template <typename T, int D>
cudaError_t run_prefill_t(const DecodeArgs &a, const T *k, const T *v, const T *qwin, int P, cudaStream_t stream,
                          unsigned long long *launches, float *S, size_t scratch_floats, int n_states, const PrefillRow *row)
{
    // `row`: the units of `a` are one batch row of a ragged batch - the tensors are padded to the longest prompt, the
    // ring slots follow the common time axis, the caller sets the step state and synchronises after the last row
    const int Ps = row ? row->kv_stride : P, shift = row ? row->shift : 0;
    const int U = a.U, G = a.G, R = a.R, C = a.C;
    // the CUDA-core scoring kernels work on the model's Gq heads per window position (rows of S); the ring keeps G
    // heads per slot, the padding heads with normaliser +inf from init_arena_kernel
    const int Rw = P < R ? P : R, rows = Rw * a.Gq;
    const bool select = P - Rw > C;
    const int n = select ? C + Rw : P;
    if (n > a.cap) return cudaErrorInvalidValue;
    // bf16 / head_dim 128 shapes score on the tensor cores (two passes over the keys, no rows x P table); the
    // others materialise the window-row logits S [rows][P] per unit and reduce them with CUDA-core kernels
    // (the arena's group must be the padded one: a context that runs the CUDA-core decode kernel keeps G as it is)
    const bool tc = !row && prefill_tc_supported(sizeof(T) == 4, D, a.Gq, R, k, P) && tc_padded_group(a.Gq) == G;
    const int Rws = row ? row->qw_stride : Rw;
    const int tc_splits = tc ? prefill_tc_splits(U, P, Rw * G) : 0;
    const size_t per_unit = tc ? prefill_tc_floats_per_unit(P, Rw, G, tc_splits) : (size_t)rows * P + P;   // floats
    if (per_unit + 1 > scratch_floats) return cudaErrorInvalidConfiguration;
    size_t ub = (scratch_floats - 1) / per_unit;
    if (ub > (size_t)U) ub = U;
    if (ub > 65535) ub = 65535;
    float *Fp = tc ? S : S + ub * (size_t)rows * P;
    float *part = S + ub * (size_t)P;                          // tensor-core path: pass-1 partials behind the scores
    int *err_word = reinterpret_cast<int *>(S + scratch_floats - 1);

    const size_t logits_smem = (size_t)(kPK * (D + 4) + kPR * (D + 4) + kPK * (kPR + 1)) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(prefill_logits_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)logits_smem);
    if (e != cudaSuccess) return e;
    const size_t init_n = max((size_t)U * a.cap, (size_t)U * R * G);
    init_arena_kernel<<<(unsigned)((init_n + 255) / 256), 256, 0, stream>>>(a);
    ++*launches;
    if (tc) {
        e = cudaMemsetAsync(err_word, 0, sizeof(int), stream);
        if (e != cudaSuccess) return e;
    }
    for (int ub0 = 0; ub0 < U; ub0 += (int)ub) {
        const int nb = min((int)ub, U - ub0);
        if (tc) {
            e = run_prefill_scores_tc(a, k, qwin, P, ub0, nb, tc_splits, Fp, part, err_word, launches, stream);
            if (e != cudaSuccess) return e;
        } else {
            prefill_logits_kernel<T, D><<<dim3((P + kPK - 1) / kPK, nb), kPT, logits_smem, stream>>>(k, qwin, S, ub0, P, Rw,
                                                                                                 a.Gq, a.scale2, Ps, Rws);
            prefill_rowstats_kernel<<<dim3(rows, nb), kPT, 0, stream>>>(S, a.ring_c, ub0, P, Rw, a.Gq, G, R, shift);
            *launches += 2;
        }
        if (select) {
            if (!tc) {
                prefill_fuse_kernel<<<dim3((P - Rw + kPT - 1) / kPT, nb), kPT, rows * sizeof(float), stream>>>(
                    S, a.ring_c, Fp, ub0, P, Rw, a.Gq, G, R, a.fusion, shift);
                ++*launches;
            }
            prefill_select_kernel<<<nb, kSelT, 0, stream>>>(Fp, a.pos, ub0, P, Rw, C, a.cap);
            ++*launches;
        }
    }
    if (!select) {
        prefill_identity_pos_kernel<<<(unsigned)(((size_t)U * n + 255) / 256), 256, 0, stream>>>(a.pos, U, n, a.cap);
        ++*launches;
    }
    constexpr int CH = D * sizeof(T) / 16;
    prefill_gather_kernel<T, D><<<dim3(U, (n * CH + 255) / 256), 256, 0, stream>>>(k, v, a, Ps, n);
    if (((uintptr_t)qwin & 15) == 0)
        prefill_ring_vec_kernel<T, D><<<dim3(U, (Rw * G * CH + 255) / 256), 256, 0, stream>>>(qwin, a, P, Rw, Rws, shift);
    else
        prefill_ring_kernel<T, D><<<U, 256, 0, stream>>>(qwin, a, P, Rw, Rws, shift);
    if (a.norm_current && select) {
        prefill_renorm_kernel<T, D><<<dim3(Rw * G, U), kPT, 0, stream>>>(a, P, Rw, n, shift);
        ++*launches;
    }
    *launches += 2;
    if (row) return cudaGetLastError();
    set_state_kernel<<<1, 32, 0, stream>>>(a.st, n_states, (long long)P, n);
    *launches += 1;
    e = cudaGetLastError();
    const cudaError_t e2 = cudaStreamSynchronize(stream);
    if (e != cudaSuccess || e2 != cudaSuccess) return e != cudaSuccess ? e : e2;
    if (tc) {       // a bounded wait of the scoring kernels that ran out
        int werr = 0;
        e = cudaMemcpy(&werr, err_word, sizeof(int), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return e;
        if (werr != 0) return cudaErrorLaunchTimeout;
    }
    return cudaSuccess;
}

cudaError_t dispatch_prefill(const DecodeArgs &a, bool f32, int D, const void *k, const void *v, const void *q_window, int P,
                             cudaStream_t stream, unsigned long long *launches, float *S, size_t scratch_floats, int n_states,
                             const PrefillRow *row = nullptr)
{
    if (f32) {
        auto kk = static_cast<const float *>(k), vv = static_cast<const float *>(v), qq = static_cast<const float *>(q_window);
        return D == 64 ? run_prefill_t<float, 64>(a, kk, vv, qq, P, stream, launches, S, scratch_floats, n_states, row)
                       : run_prefill_t<float, 128>(a, kk, vv, qq, P, stream, launches, S, scratch_floats, n_states, row);
    }
    auto kk = static_cast<const __nv_bfloat16 *>(k), vv = static_cast<const __nv_bfloat16 *>(v),
         qq = static_cast<const __nv_bfloat16 *>(q_window);
    return D == 64 ? run_prefill_t<__nv_bfloat16, 64>(a, kk, vv, qq, P, stream, launches, S, scratch_floats, n_states, row)
                   : run_prefill_t<__nv_bfloat16, 128>(a, kk, vv, qq, P, stream, launches, S, scratch_floats, n_states, row);
}

// ---- scratch of mkv_prefill_static -------------------------------------------------------------------------
// A fixed device array that every GPU loading this library holds until the process exits.  16 MiB: one unit of a
// 4096-token prompt with R*G = 128 window rows needs 2.1 MB, so the units go through it a few at a time.
constexpr size_t kStaticScratchFloats = (size_t)4 << 20;
static __device__ __align__(256) float g_prefill_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
static float *g_scratch_addr[kMaxDevices];   // device address of the array, per device ordinal
static std::mutex g_scratch_mutex;

// The array's name is only a host-side handle here; a kernel needs its device address, which the runtime hands out
// per device.  Looked up once per device, with that device current.
cudaError_t static_scratch_address(int device, float **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (dev != device) return cudaErrorInvalidDevice;          // the context lives on another device than the current one
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        float *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_prefill_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

cudaError_t run_prefill(const DecodeArgs &a, bool f32, int D, const void *k, const void *v, const void *q_window, int P,
                        cudaStream_t stream, unsigned long long *launches, PrefillScratch *scratch, int n_states,
                        const PrefillRow *row)
{
    const int Rw = P < a.R ? P : a.R;
    const bool tc = !row && prefill_tc_supported(f32, D, a.Gq, a.R, k, P) && tc_padded_group(a.Gq) == a.G;
    const size_t per_unit = (tc ? prefill_tc_floats_per_unit(P, Rw, a.G, prefill_tc_splits(a.U, P, Rw * a.G))
                                : (size_t)Rw * a.G * P + P) * sizeof(float);
    size_t ub = ((size_t)1 << 30) / per_unit;
    if (ub < 1) ub = 1;
    if (ub > (size_t)a.U) ub = a.U;
    if (ub > 65535) ub = 65535;
    const size_t need = ub * per_unit + sizeof(float);          // + the error word of the scoring kernels
    // The scratch belongs to the context and is kept until the context is destroyed: it only grows.
    // (Allocating and freeing it around every prompt put a cudaFree of up to 1 GiB right in front
    // of the first decode launches.)
    if (scratch->bytes < need) {
        if (scratch->ptr) cudaFree(scratch->ptr);
        scratch->ptr = nullptr;
        scratch->bytes = 0;
        const cudaError_t e = cudaMalloc(&scratch->ptr, need);
        if (e != cudaSuccess) { scratch->ptr = nullptr; return e; }
        scratch->bytes = need;
    }
    return dispatch_prefill(a, f32, D, k, v, q_window, P, stream, launches, static_cast<float *>(scratch->ptr),
                            scratch->bytes / sizeof(float), n_states, row);
}

cudaError_t launch_set_state(DevState *st, int n_states, long long t, int n, cudaStream_t stream)
{
    set_state_kernel<<<1, 32, 0, stream>>>(st, n_states, t, n);
    return cudaGetLastError();
}

namespace {
// rows_dst / rows_src: the states' per-row fills ([2][B] ints per state, see DecodeArgs::row_n), or nullptr
__global__ void copy_state_kernel(DevState *dst, int n_dst, const DevState *src, int *rows_dst, const int *rows_src,
                                  int row_ints)
{
    const DevState s = *src;
    __syncthreads();            // src may be one of the destinations
    for (int i = threadIdx.x; i < n_dst; i += blockDim.x) { dst[i] = s; dst[i].done = 0; }
    if (rows_dst != nullptr && rows_dst != rows_src)
        for (int i = threadIdx.x; i < n_dst * row_ints; i += blockDim.x) rows_dst[i] = rows_src[i % row_ints];
}
}  // namespace

cudaError_t launch_copy_state(DevState *dst, int n_dst, const DevState *src, cudaStream_t stream, int *rows_dst,
                              const int *rows_src, int row_ints)
{
    copy_state_kernel<<<1, 64, 0, stream>>>(dst, n_dst, src, rows_dst, rows_src, row_ints);
    return cudaGetLastError();
}

size_t prefill_static_max_floats() { return kStaticScratchFloats; }

cudaError_t run_prefill_static(const DecodeArgs &a, bool f32, int D, const void *k, const void *v, const void *q_window,
                               int P, cudaStream_t stream, unsigned long long *launches, int device, int n_states)
{
    float *S = nullptr;
    const cudaError_t e = static_scratch_address(device, &S);
    if (e != cudaSuccess) return e;
    return dispatch_prefill(a, f32, D, k, v, q_window, P, stream, launches, S, kStaticScratchFloats, n_states);
}

}  // namespace mkv
