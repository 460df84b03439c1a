// Host-callable launchers of the MorphKV kernels (internal to the library).
#pragma once

#include "mkv_common.cuh"

namespace mkv {

// CUDA-core decode step (any supported shape).  `a.splits` CTAs per unit.
cudaError_t launch_decode_simt(const DecodeArgs &a, bool f32, int D, cudaStream_t stream);
int simt_default_splits(int U, int cap);

// Coarse-grained eviction (evict_interval > 1): drops everything beyond the top C after a step that scored and
// restores the dense prefix of C + R slots; a no-op after the other steps.  Launched after every decode step.
cudaError_t launch_compact(const DecodeArgs &a, bool f32, int D, cudaStream_t stream);

// Tensor-core (tcgen05) decode step: bf16, head_dim 128, GQA group padded to {1,2,4,8,16}.  A window of up to
// 256 ring rows (R * padded group) is one MMA operand; a larger one is cut into tc_ring_chunks() chunks of equal
// width, and a unit then appears in the kernel's schedule once per chunk (U * chunks "virtual units": pass that
// count to tc_grid() and tc_partials_per_unit()).  The plan holds the TMA tensor maps of a context's arena and
// the launch geometry; `a.splits` must be tc_partials_per_unit() of the grid (every CTA that holds tiles of a
// unit leaves one partial).
bool tc_shape_supported(bool f32, int D, int G, int R);
int tc_padded_group(int G);
int tc_ring_chunks(int G, int R);
int tc_grid(int U, int cap, int splits_hint, int n_sm);
int tc_partials_per_unit(int U, int cap, int grid);
struct TcPlan;
// `prefetch`: CTAs ask for the first tiles of their range into L2 while the previous launch drains.
cudaError_t tc_plan_create(TcPlan **plan, const DecodeArgs &a, int grid, unsigned long long wait_limit_cycles, bool prefetch,
                           char *err, size_t err_len);
void tc_plan_destroy(TcPlan *plan);
cudaError_t launch_decode_tc(TcPlan *plan, const DecodeArgs &a, cudaStream_t stream);

// Prompt phase: fills the arena (K, V, pos, ring) and the n_states step states at a.st from a prompt of P
// tokens.  `a` supplies the arena pointers and shape; q/k_new/v_new/out are ignored.
// *launches is advanced per kernel launched.
// Device scratch of the prompt phase, owned by the context (allocated on first use, grown when a
// longer prompt needs more, released with the context).
struct PrefillScratch {
    void *ptr;
    size_t bytes;
};
// One batch row of a batch whose prompts have different lengths: `a` covers the row's units of one layer, k / v /
// q_window point at the row's first unit inside tensors padded to the longest prompt (kv_stride tokens per unit,
// qw_stride window entries per head), and the row is `shift` positions behind the longest on the context's common
// time axis, which assigns the ring slots.  Such a call leaves the step state alone and does not synchronise.
struct PrefillRow {
    int kv_stride, qw_stride, shift;
};
cudaError_t run_prefill(const DecodeArgs &a, bool f32, int D, const void *k, const void *v, const void *q_window,
                        int P, cudaStream_t stream, unsigned long long *launches, PrefillScratch *scratch, int n_states,
                        const PrefillRow *row = nullptr);
cudaError_t launch_set_state(DevState *st, int n_states, long long t, int n, cudaStream_t stream);

// Tensor-core scoring of the prompt phase (mkv_prefill_tc.cu): two passes over the prompt keys, window-row
// normalisers into ring_c and fused scores of the older tokens into Fp [nb][P].
bool prefill_tc_supported(bool f32, int D, int G, int R, const void *k, int P);
int prefill_tc_splits(int units_in_batch, int P, int window_rows);
size_t prefill_tc_floats_per_unit(int P, int Rw, int G, int splits);
cudaError_t run_prefill_scores_tc(const DecodeArgs &a, const void *k, const void *qwin, int P, int ub0, int nb, int splits,
                                  float *Fp, float *part, int *err, unsigned long long *launches, cudaStream_t stream);

// The same prompt phase with its scratch in a fixed device array of prefill_static_max_floats()
// floats instead of a temporary allocation; cudaErrorInvalidConfiguration if one unit's
// (R*G + 1) * P floats do not fit.
size_t prefill_static_max_floats();
cudaError_t run_prefill_static(const DecodeArgs &a, bool f32, int D, const void *k, const void *v, const void *q_window,
                               int P, cudaStream_t stream, unsigned long long *launches, int device, int n_states);

// Stored-profile mode (bf16, head_dim 128, tensor-core kernel): the fused scores of a policy step from the profile
// table into a.F (a no-op on other steps; launched in front of the decode kernel), and the table after the prompt
// phase (the arena's ring, K rows and positions must be in place; the table must have been cleared).
cudaError_t launch_profile_fuse(const DecodeArgs &a, cudaStream_t stream);
cudaError_t launch_prefill_profile(const DecodeArgs &a, int n, long long P, cudaStream_t stream);

// Copies one step state over n_dst others (the whole-stack state and the per-layer states are brought level when
// a context switches between whole-stack and per-layer calls).
cudaError_t launch_copy_state(DevState *dst, int n_dst, const DevState *src, cudaStream_t stream, int *rows_dst = nullptr,
                              const int *rows_src = nullptr, int row_ints = 0);

}  // namespace mkv
