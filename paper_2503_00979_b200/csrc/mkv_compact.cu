// Coarse-grained eviction (the paper's appendix on running the policy every T-th step): the decode
// step that scored has appended its token like any other step and left the final fused score of
// every slot in F (-1 for the slots of the recent window).  This launch then applies Eq. 7 once:
// it drops the E = n - (C + R) lowest-ranked candidates (lower fused score first, on equal scores
// the later position first, so that the lower position is the one kept) and moves the survivors
// that sit beyond slot C + R into the freed slots, which restores a dense prefix of C + R slots.
// One CTA of 1024 threads per unit, each thread holding a few slots' rank keys; launched after the
// decode steps that ran the policy, and a no-op unless the device state says a compaction is pending.
#include "mkv_common.cuh"
#include "mkv_kernels.h"

namespace mkv {

namespace {

constexpr int kCT = 1024;         // threads per CTA

// KPT slots per thread, held in registers (indices are compile-time constants after unrolling)
template <typename T, int D, int KPT>
__global__ void __launch_bounds__(kCT) compact_kernel(DecodeArgs a)
{
    __shared__ unsigned long long red_key[kCT / 32];
    __shared__ int red_slot[kCT / 32];
    __shared__ int ev_slot[64];          // evicted slots, in eviction order
    __shared__ int holes[64], movers[64];
    __shared__ int n_holes;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.x;
    const bool pending = a.st->compact != 0;
    const int n = a.st->n;                       // tokens cached after the step's append
    const int keep = a.C + a.R;
    const int E = n - keep;
    if (pending && E > 0) {
        int *pos = a.pos + (size_t)u * a.cap;
        float *F = a.F + (size_t)u * a.cap;
        // every thread's candidates as rank keys (window slots carry F = -1 and never compete)
        unsigned long long key[KPT];
#pragma unroll
        for (int i = 0; i < KPT; ++i) {
            const int k = tid + i * kCT;
            unsigned long long v = ~0ull;
            if (k < n) {
                const float f = F[k];
                if (f >= 0.f) v = rank_key(__float_as_uint(f), pos[k]);
            }
            key[i] = v;
        }
        for (int e = 0; e < E; ++e) {
            // lowest rank key of the block: thread, warp, then the first warp over the warps' minima
            unsigned long long best = ~0ull;
            int bslot = -1;
#pragma unroll
            for (int i = 0; i < KPT; ++i)
                if (key[i] < best) { best = key[i]; bslot = tid + i * kCT; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
                const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
                if (ok < best) { best = ok; bslot = os; }
            }
            if (lane == 0) { red_key[warp] = best; red_slot[warp] = bslot; }
            __syncthreads();
            if (warp == 0) {
                best = red_key[lane]; bslot = red_slot[lane];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
                    const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
                    if (ok < best) { best = ok; bslot = os; }
                }
                if (lane == 0) ev_slot[e] = bslot;
            }
            __syncthreads();
            bslot = ev_slot[e];
            if (bslot >= 0 && (bslot % kCT) == tid) {       // its owner retires it
#pragma unroll
                for (int i = 0; i < KPT; ++i)
                    if (i == bslot / kCT) key[i] = ~0ull;
            }
        }
        // holes: evicted slots inside the kept prefix; movers: surviving slots beyond it (both ascending)
        if (tid == 0) {
            int nh = 0;
            for (int e = 0; e < E; ++e)
                if (ev_slot[e] >= 0 && ev_slot[e] < keep) holes[nh++] = ev_slot[e];
            for (int i = 1; i < nh; ++i) {          // insertion sort of at most T entries
                const int v = holes[i];
                int j = i - 1;
                while (j >= 0 && holes[j] > v) { holes[j + 1] = holes[j]; --j; }
                holes[j + 1] = v;
            }
            int nm = 0;
            for (int k = keep; k < n; ++k) {
                bool gone = false;
                for (int e = 0; e < E; ++e) gone |= ev_slot[e] == k;
                if (!gone) movers[nm++] = k;
            }
            n_holes = nh < nm ? nh : nm;            // equal by construction
        }
        __syncthreads();
        const int nh = n_holes;
        T *K = static_cast<T *>(a.K) + (size_t)u * a.cap * D;
        T *V = static_cast<T *>(a.V) + (size_t)u * a.cap * D;
        for (int idx = tid; idx < nh * D; idx += kCT) {
            const int i = idx / D, c = idx % D;
            K[(size_t)holes[i] * D + c] = K[(size_t)movers[i] * D + c];
            V[(size_t)holes[i] * D + c] = V[(size_t)movers[i] * D + c];
        }
        __syncthreads();
        if (tid < nh) { pos[holes[tid]] = pos[movers[tid]]; F[holes[tid]] = F[movers[tid]]; }
        __syncthreads();
        for (int k = keep + tid; k < n; k += kCT) { pos[k] = -1; F[k] = 0.f; }
        if (tid == 0) a.evicted_pos[u] = -1;
    }
    // the last CTA publishes the new fill (all CTAs have read the state by then)
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(&a.st->done, 1u) == gridDim.x - 1) {
            if (pending && E > 0) a.st->n = keep;
            a.st->compact = 0;
            a.st->done = 0;
            __threadfence();
        }
    }
}

}  // namespace

template <typename T, int D>
static void launch_compact_t(const DecodeArgs &a, cudaStream_t stream)
{
    const int per = (a.cap + kCT - 1) / kCT;
    if (per <= 2) compact_kernel<T, D, 2><<<a.U, kCT, 0, stream>>>(a);
    else if (per <= 4) compact_kernel<T, D, 4><<<a.U, kCT, 0, stream>>>(a);
    else if (per <= 8) compact_kernel<T, D, 8><<<a.U, kCT, 0, stream>>>(a);
    else compact_kernel<T, D, 16><<<a.U, kCT, 0, stream>>>(a);
}

cudaError_t launch_compact(const DecodeArgs &a, bool f32, int D, cudaStream_t stream)
{
    if (a.T > 64 || (a.cap + kCT - 1) / kCT > 16) return cudaErrorInvalidConfiguration;
    if (f32) {
        if (D == 64) launch_compact_t<float, 64>(a, stream); else launch_compact_t<float, 128>(a, stream);
    } else {
        if (D == 64) launch_compact_t<__nv_bfloat16, 64>(a, stream); else launch_compact_t<__nv_bfloat16, 128>(a, stream);
    }
    return cudaGetLastError();
}

}  // namespace mkv
