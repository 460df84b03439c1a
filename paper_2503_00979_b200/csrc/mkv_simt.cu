// CUDA-core decode kernel: any dtype (bf16 / f32), head_dim 64 or 128, any GQA group and
// window size.  It is the kernel of the f32 mode and of shapes the tensor-core kernel does
// not take, and serves as an on-device cross-check of that kernel.
//
// One CTA handles one (unit, split): a contiguous range of the unit's cached keys.
//   K phase  for every key of the range: log2-domain logits against all R*G ring rows
//            (the new query standing in for the row that leaves the window); ring rows
//            other than the new one turn into frozen soft-max weights
//            exp2(s - c_row), are summed over the GQA group and fused over the window
//            (Eq. 4-6, Algorithm 1); the new row's raw logits are kept for the epilogue.
//   V phase  soft-max of the new row over the range and its weighted sum of V (Eq. 1).
//   The CTA that finishes a unit last merges the splits, selects and appends (Eq. 7).
#include "mkv_common.cuh"
#include "mkv_kernels.h"

namespace mkv {

constexpr int kThreads = 256;
constexpr int kTK = 32;   // keys per tile
constexpr int kSB = 64;   // ring rows per scoring sub-block

template <typename T> struct Pad;
template <> struct Pad<float> { static constexpr int q = 4; };
template <> struct Pad<__nv_bfloat16> { static constexpr int q = 8; };

__device__ __forceinline__ void load4(const float *p, float (&o)[4])
{
    const float4 v = *reinterpret_cast<const float4 *>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16 *p, float (&o)[4])
{
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
}
__device__ __forceinline__ void copy4(float *d, const float *s)
{
    *reinterpret_cast<float4 *>(d) = *reinterpret_cast<const float4 *>(s);
}
__device__ __forceinline__ void copy4(__nv_bfloat16 *d, const __nv_bfloat16 *s)
{
    *reinterpret_cast<uint2 *>(d) = *reinterpret_cast<const uint2 *>(s);
}

struct SimtSmem {
    size_t q_off, c_off, k_off, s_off, f_off, p_off, misc_off, total;
};

// chunk_rows = ring rows resident at a time
template <typename T, int D>
__host__ __device__ inline SimtSmem simt_smem_layout(int chunk_rows, int G)
{
    SimtSmem L;
    size_t o = 0;
    L.q_off = o; o += (size_t)chunk_rows * (D + Pad<T>::q) * sizeof(T); o = (o + 15) & ~(size_t)15;
    L.c_off = o; o += (size_t)chunk_rows * sizeof(float); o = (o + 15) & ~(size_t)15;
    L.k_off = o; o += (size_t)kTK * (D + 4) * sizeof(float);
    L.s_off = o; o += (size_t)kTK * (kSB + 1) * sizeof(float); o = (o + 15) & ~(size_t)15;
    L.f_off = o; o += (size_t)kTK * sizeof(float);
    L.p_off = o; o += (size_t)G * kThreads * sizeof(float);
    L.misc_off = o; o += 384 * sizeof(float);
    L.total = o;
    return L;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) decode_simt_kernel(const __grid_constant__ DecodeArgs a, const int chunk_rs)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.G, R = a.R;
    const int u = blockIdx.x / a.splits, sp = blockIdx.x % a.splits;
    const long long t = a.st->t;
    const int n = a.st->n;
    const int steps_done = a.st->steps;
    const bool evict_all = step_scores(t, n, steps_done, R, a.C, a.T);
    // the unit's own fill and policy decision (they differ from the uniform ones only between batch rows whose
    // prompts had different lengths); the splits are laid out over the largest fill
    const UnitStep us = unit_step(a, u, t, n, steps_done, evict_all);
    const bool evict = us.evict;
    int active;
    const int per = split_len(n, a.splits, kTK, &active);
    const int k0 = sp * per, k1 = min(us.n, k0 + per);

    const SimtSmem L = simt_smem_layout<T, D>(chunk_rs * G, G);
    T *Qs = reinterpret_cast<T *>(smem_raw + L.q_off);
    float *cs = reinterpret_cast<float *>(smem_raw + L.c_off);
    float *Ks = reinterpret_cast<float *>(smem_raw + L.k_off);
    float *Ssm = reinterpret_cast<float *>(smem_raw + L.s_off);
    float *Facc = reinterpret_cast<float *>(smem_raw + L.f_off);
    float *Psm = reinterpret_cast<float *>(smem_raw + L.p_off);
    float *misc = reinterpret_cast<float *>(smem_raw + L.misc_off);
    __shared__ int is_last;
    constexpr int QS = D + Pad<T>::q, KS = D + 4, C4 = D / 4;

    if (k0 < n) {
        const int rs_new = (int)(t % R);
        const T *q = static_cast<const T *>(a.q) + (size_t)u * G * D;
        const T *ring_q = static_cast<const T *>(a.ring_q) + (size_t)u * R * G * D;
        const float *ring_c = a.ring_c + (size_t)u * R * G;
        const T *Ku = static_cast<const T *>(a.K) + (size_t)u * a.cap * D;
        const T *Vu = static_cast<const T *>(a.V) + (size_t)u * a.cap * D;
        float *s_new = a.s_new + (size_t)u * G * a.cap;
        float *Fu = a.F + (size_t)u * a.cap;
        // without an eviction only the new row is needed (Eq. 1); scoring is skipped
        const int rs_begin = evict ? 0 : rs_new, rs_end = evict ? R : rs_new + 1;
        const int sbr = max(1, kSB / G);          // ring slots per sub-block
        const int tx = tid & 15, ty = tid >> 4;   // 4 rows (tx + 16 i) x 2 keys (ty, ty + 16) per thread

        // ---------------- K phase ----------------
        for (int cr0 = rs_begin; cr0 < rs_end; cr0 += chunk_rs) {
            const int cr1 = min(rs_end, cr0 + chunk_rs);
            const int nrows = (cr1 - cr0) * G;
            __syncthreads();
            for (int idx = tid; idx < nrows * C4; idx += kThreads) {
                const int row = idx / C4, c4 = idx % C4;
                const int rslot = cr0 + row / G, g = row % G;
                const T *src = (rslot == rs_new) ? q + (size_t)g * D : ring_q + ((size_t)rslot * G + g) * D;
                copy4(Qs + (size_t)row * QS + c4 * 4, src + c4 * 4);
            }
            for (int row = tid; row < nrows; row += kThreads) {
                const int rslot = cr0 + row / G;
                cs[row] = (rslot == rs_new) ? 0.f : ring_c[(size_t)cr0 * G + row];
            }
            __syncthreads();
            for (int kt = k0; kt < k1; kt += kTK) {
                for (int idx = tid; idx < kTK * C4; idx += kThreads) {
                    const int key = idx / C4, c4 = idx % C4;
                    float v[4] = {0.f, 0.f, 0.f, 0.f};
                    if (kt + key < k1) load4(Ku + (size_t)(kt + key) * D + c4 * 4, v);
                    *reinterpret_cast<float4 *>(Ks + key * KS + c4 * 4) = make_float4(v[0], v[1], v[2], v[3]);
                }
                if (tid < kTK) Facc[tid] = 0.f;
                __syncthreads();
                for (int sb0 = 0; sb0 < cr1 - cr0; sb0 += sbr) {
                    const int nrs_sb = min(sbr, cr1 - cr0 - sb0);
                    const int nrows_sb = nrs_sb * G, rowbase = sb0 * G;
                    float acc[2][4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) { acc[0][i] = 0.f; acc[1][i] = 0.f; }
                    const T *qrow[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rl = tx + 16 * i;
                        qrow[i] = Qs + (size_t)(rowbase + (rl < nrows_sb ? rl : 0)) * QS;
                    }
                    const float *ka = Ks + ty * KS, *kb = Ks + (ty + 16) * KS;
#pragma unroll 4
                    for (int dd = 0; dd < D; dd += 4) {
                        const float4 x = *reinterpret_cast<const float4 *>(ka + dd);
                        const float4 y = *reinterpret_cast<const float4 *>(kb + dd);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float qv[4];
                            load4(qrow[i] + dd, qv);
                            acc[0][i] += x.x * qv[0] + x.y * qv[1] + x.z * qv[2] + x.w * qv[3];
                            acc[1][i] += y.x * qv[0] + y.y * qv[1] + y.z * qv[2] + y.w * qv[3];
                        }
                    }
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        const int key = ty + 16 * kk;
                        const bool kvalid = kt + key < k1;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int rl = tx + 16 * i;
                            if (rl >= nrows_sb) continue;
                            const int row = rowbase + rl;
                            const int rslot = cr0 + row / G;
                            const float s2 = acc[kk][i] * a.scale2;
                            float w = 0.f;
                            if (rslot == rs_new) {
                                if (kvalid) s_new[(size_t)(row % G) * a.cap + kt + key] = s2;
                            } else if (kvalid) {
                                w = exp2f(s2 - cs[row]);     // weight the row assigned when generated
                            }
                            Ssm[key * (kSB + 1) + rl] = w;
                        }
                    }
                    __syncthreads();
                    {   // sum over the GQA group, fuse over the window rows of this sub-block
                        const int key = tid >> 3, l8 = tid & 7;
                        float f = 0.f;
                        for (int r = l8; r < nrs_sb; r += 8) {
                            float S = 0.f;
                            for (int g = 0; g < G; ++g) S += Ssm[key * (kSB + 1) + r * G + g];
                            f = fuse(a.fusion, f, S);
                        }
#pragma unroll
                        for (int o = 4; o > 0; o >>= 1) f = fuse(a.fusion, f, __shfl_xor_sync(0xffffffffu, f, o));
                        if (l8 == 0) Facc[key] = fuse(a.fusion, Facc[key], f);
                    }
                    __syncthreads();
                }
                if (evict && tid < kTK && kt + tid < k1) {
                    const float f = Facc[tid];
                    Fu[kt + tid] = (cr0 == rs_begin) ? f : fuse(a.fusion, Fu[kt + tid], f);
                }
                __syncthreads();
            }
        }

        // ---------------- V phase (Eq. 1 over this split) ----------------
        float *mloc = misc, *lloc = misc + kMaxGroup, *red = misc + 2 * kMaxGroup;   // red[8]
        for (int g = 0; g < G; ++g) {
            float mx = -INFINITY;
            for (int k = k0 + tid; k < k1; k += kThreads) mx = fmaxf(mx, s_new[(size_t)g * a.cap + k]);
            mx = warp_max(mx);
            if (lane == 0) red[warp] = mx;
            __syncthreads();
            if (tid == 0) {
                float m = red[0];
                for (int w = 1; w < kThreads / 32; ++w) m = fmaxf(m, red[w]);
                mloc[g] = m;
            }
            __syncthreads();
        }
        constexpr int kParts = kThreads / D;
        const int dcol = tid % D, part = tid / D;
        float oacc[kMaxGroup], lsum[kMaxGroup];
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) { oacc[g] = 0.f; lsum[g] = 0.f; }
        for (int c0 = k0; c0 < k1; c0 += kThreads) {
            const int kk = c0 + tid;
#pragma unroll
            for (int g = 0; g < kMaxGroup; ++g) {
                if (g < G) {
                    const float p = kk < k1 ? exp2f(s_new[(size_t)g * a.cap + kk] - mloc[g]) : 0.f;
                    Psm[g * kThreads + tid] = p;
                    lsum[g] += p;
                }
            }
            __syncthreads();
            const int cnt = min(kThreads, k1 - c0);
            for (int j = part; j < cnt; j += kParts) {
                const float v = ldf(Vu + (size_t)(c0 + j) * D + dcol);
#pragma unroll
                for (int g = 0; g < kMaxGroup; ++g)
                    if (g < G) oacc[g] += Psm[g * kThreads + j] * v;
            }
            __syncthreads();
        }
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
            if (g < G) {
                const float s = warp_sum(lsum[g]);
                if (lane == 0) red[warp] = s;
                __syncthreads();
                if (tid == 0) {
                    float l = 0.f;
                    for (int w = 0; w < kThreads / 32; ++w) l += red[w];
                    lloc[g] = l;
                }
                __syncthreads();
                Psm[g * kThreads + tid] = oacc[g];    // tid == part * D + dcol
            }
        }
        __syncthreads();
        float *pml = a.part_ml + ((size_t)u * a.splits + sp) * G * 2;
        float *po = a.part_o + ((size_t)u * a.splits + sp) * G * D;
        for (int idx = tid; idx < G * D; idx += kThreads) {
            const int g = idx / D, dd = idx % D;
            float o = 0.f;
            for (int p = 0; p < kParts; ++p) o += Psm[g * kThreads + p * D + dd];
            po[idx] = o;
        }
        if (tid < G) { pml[tid * 2] = mloc[tid]; pml[tid * 2 + 1] = lloc[tid]; }

        // ---------------- last split of the unit finalises it ----------------
        __threadfence();
        __syncthreads();
        if (tid == 0) is_last = (atomicAdd(&a.ticket[u], 1) == active - 1);
        __syncthreads();
        if (is_last) {
            __threadfence();
            finalize_unit<T, D, 0>(a, u, t, us.n, active, evict, misc + 64, tid, kThreads, 0, us.shift);
        }
    }
    finish_cta(a, t, n, evict_all);
}

template <typename T, int D>
static cudaError_t launch_simt_t(const DecodeArgs &a, cudaStream_t stream)
{
    // ring rows kept resident: as many window slots as fit beside the fixed buffers
    const size_t budget = 200 * 1024;
    const size_t fixed = simt_smem_layout<T, D>(0, a.G).total;
    const size_t per_rs = (size_t)a.G * ((D + Pad<T>::q) * sizeof(T) + sizeof(float)) + 32;
    int chunk_rs = (int)((budget - fixed) / per_rs);
    if (chunk_rs < 1) return cudaErrorInvalidConfiguration;
    if (chunk_rs > a.R) chunk_rs = a.R;
    const size_t smem = simt_smem_layout<T, D>(chunk_rs * a.G, a.G).total;
    auto kern = decode_simt_kernel<T, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<a.U * a.splits, kThreads, smem, stream>>>(a, chunk_rs);
    return cudaGetLastError();
}

cudaError_t launch_decode_simt(const DecodeArgs &a, bool f32, int D, cudaStream_t stream)
{
    if (f32) return D == 64 ? launch_simt_t<float, 64>(a, stream) : launch_simt_t<float, 128>(a, stream);
    return D == 64 ? launch_simt_t<__nv_bfloat16, 64>(a, stream) : launch_simt_t<__nv_bfloat16, 128>(a, stream);
}

int simt_default_splits(int U, int cap)
{
    // about two waves of 148 SMs, but at least 128 keys per split
    int s = (2 * 148 + U - 1) / U;
    const int max_s = (cap + 127) / 128;
    if (s > max_s) s = max_s;
    return s < 1 ? 1 : s;
}

}  // namespace mkv
