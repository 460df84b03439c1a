// Stored-profile mode: the attention profiles of the window tokens are kept as a table beside the KV cache, the way
// the paper's implementation keeps them (Implementation paragraph), instead of being recomputed from the stored
// window queries.  prof[u][r][k] is the weight, summed over the GQA group, that the window token of ring slot r
// gave to the token in cache slot k at the step that generated it (0 where it never saw that token).  Per policy
// step the table is read once (R * n floats per unit) and fused into F (Eq. 4-6); the decode kernel then attends
// only, and its epilogue writes the new token's row and clears the column of the slot that changes hands.
// A trade of bytes for arithmetic: it pays where the recomputation is bound by exponentials (wide windows).
#include "mkv_common.cuh"
#include "mkv_kernels.h"

namespace mkv {

namespace {

constexpr int kFT = 256;

// F[k] = sum or max over the window rows of prof[r][k], without the row of the token that leaves the window on
// this step (ring slot t % R, which the new token's row replaces).
__global__ void __launch_bounds__(kFT) profile_fuse_kernel(DecodeArgs a)
{
    const long long t = a.st->t;
    const int n = a.st->n;
    if (!step_scores(t, n, a.st->steps, a.R, a.C, a.T)) return;
    const int u = blockIdx.y, k = blockIdx.x * kFT + threadIdx.x;
    if (k >= n) return;
    const int rs = (int)(t % a.R);
    const float *p = a.prof + (size_t)u * a.R * a.cap + k;
    float F = 0.f;
    int r = 0;
    for (; r + 8 <= a.R; r += 8) {          // eight rows in flight
        float w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = __ldcs(p + (size_t)(r + i) * a.cap);
#pragma unroll
        for (int i = 0; i < 8; ++i) F = fuse(a.fusion, F, r + i == rs ? 0.f : w[i]);
    }
    for (; r < a.R; ++r) F = fuse(a.fusion, F, r == rs ? 0.f : __ldcs(p + (size_t)r * a.cap));
    a.F[(size_t)u * a.cap + k] = F;
}

// The table after the prompt phase: every filled ring slot's profile over the kept tokens, from the arena as it
// stands (ring queries and their normalisers, kept K rows and their positions).  One CTA per (ring slot, unit).
template <int D>
__global__ void __launch_bounds__(kFT) prefill_profile_kernel(DecodeArgs a, int n, long long P)
{
    __shared__ float qs[kMaxGroup * D];
    __shared__ float cs[kMaxGroup];
    const int r = blockIdx.x, u = blockIdx.y, G = a.G;
    const float *c = a.ring_c + ((size_t)u * a.R + r) * G;
    // the position of the token in ring slot r: the latest p < P with p % R == r (negative: the slot is empty)
    const long long rpos = P - 1 - ((P - 1 - r) % a.R + a.R) % a.R;
    float *row = a.prof + ((size_t)u * a.R + r) * a.cap;
    if (rpos < 0 || rpos < P - a.R) return;                 // (the table was cleared beforehand)
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(a.ring_q) + ((size_t)u * a.R + r) * G * D;
    for (int i = threadIdx.x; i < G * D; i += kFT) qs[i] = __bfloat162float(q[i]);
    if (threadIdx.x < G) cs[threadIdx.x] = c[threadIdx.x];
    __syncthreads();
    const __nv_bfloat16 *K = static_cast<const __nv_bfloat16 *>(a.K) + (size_t)u * a.cap * D;
    const int *pos = a.pos + (size_t)u * a.cap;
    for (int k = threadIdx.x; k < n; k += kFT) {
        float w = 0.f;
        if ((long long)pos[k] <= rpos) {
            const uint4 *kr = reinterpret_cast<const uint4 *>(K + (size_t)k * D);
            float acc[kMaxGroup];
            for (int g = 0; g < G; ++g) acc[g] = 0.f;
            for (int ch = 0; ch < D / 8; ++ch) {
                const uint4 kv = kr[ch];
                const uint32_t *kw = reinterpret_cast<const uint32_t *>(&kv);
                float kf[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) { kf[2 * e] = __uint_as_float(kw[e] << 16); kf[2 * e + 1] = __uint_as_float(kw[e] & 0xffff0000u); }
                for (int g = 0; g < G; ++g) {
                    const float *qg = qs + g * D + ch * 8;
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[g] += qg[e] * kf[e];
                }
            }
            for (int g = 0; g < G; ++g) w += cs[g] < INFINITY ? exp2f(acc[g] * a.scale2 - cs[g]) : 0.f;
        }
        row[k] = w;
    }
}

}  // namespace

cudaError_t launch_profile_fuse(const DecodeArgs &a, cudaStream_t stream)
{
    profile_fuse_kernel<<<dim3((a.cap + kFT - 1) / kFT, a.U), kFT, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_prefill_profile(const DecodeArgs &a, int n, long long P, cudaStream_t stream)
{
    prefill_profile_kernel<128><<<dim3(a.R, a.U), kFT, 0, stream>>>(a, n, P);
    return cudaGetLastError();
}

}  // namespace mkv
