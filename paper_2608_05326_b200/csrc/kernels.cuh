// Host-callable launchers of the table, page and combine kernels (definitions in the .cu files).
#pragma once

#include "common.cuh"

namespace qevict {

struct KernelArgs {
  Geometry geo;
  State st;
  int unit0;    // first unit of this call
  int n_units;  // units of this call
  int mig_parity;  // which of the call's two migration-queue counters this routing event uses
#ifdef QEVICT_TRACE
  unsigned long long* trace;  // this call's block of the kernel timeline
#endif
};

// cache set-up: the rotation table of pre-RoPE keys (nothing to do when rope_base is 0)
cudaError_t launch_rope_table(const Geometry& g, const State& st, cudaStream_t s);
// prompt keys [rows][ctx][d] (pre-RoPE) -> rotated for positions 0 .. ctx-1 (prefill scoring with pre-RoPE keys)
cudaError_t launch_rope_rotate_prompt(const Geometry& g, const void* k, void* out, long rows, int ctx, cudaStream_t s);

// decode step ---------------------------------------------------------------------------------------
// A0: append one token per unit to its open window (opens one first if needed, zeroing the page).
// q_src / q_dst (optional): the kernel also copies the call's queries from page-locked host memory into device memory.
cudaError_t launch_append(const KernelArgs& a, const void* k_new, const void* v_new, cudaStream_t s,
                          const void* q_src = nullptr, void* q_dst = nullptr);
// A2: merge the split partials into `out`, add each window's mass to its score in fixed head order.
cudaError_t launch_combine(const KernelArgs& a, int n_splits, int e_bound, void* out, cudaStream_t s);

// routing event ---------------------------------------------------------------------------------------
// P0 (first half): every prompt window becomes an aged candidate with the given score.
cudaError_t launch_prefill_init(const KernelArgs& a, int n_prompt_windows, const float* scores, cudaStream_t s);
// key-norm ranking: scores of the prompt windows = minus the mean key norm (k: [units][H_kv][ctx][d])
cudaError_t launch_key_norm_scores(const KernelArgs& a, const void* k_prompt, int ctx, int n_prompt_windows, cudaStream_t s);
// A3 + A4 + A7: rank, assign tiers, release / allocate pages, build migration lists and the work list.
cudaError_t launch_route(const KernelArgs& a, int prefill, int sort_capacity, cudaStream_t s);
// A5 + A6: quantize the windows of the quantization list (source: their full-precision page, or the
// prompt) and dequantize the windows of the promotion list into their new full-precision page; a
// promotion that takes over the page a quantization reads runs after it in the same CTA.
cudaError_t launch_migrate(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx, int max_items,
                           cudaStream_t s);
// P0 (second half): copy the prompt windows of the copy list into their full-precision page.
cudaError_t launch_copy_prompt(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx,
                               int max_items, cudaStream_t s);

// export ------------------------------------------------------------------------------------------------
cudaError_t launch_export_fp_page(const KernelArgs& a, int unit, int page, void* k_out, void* v_out, cudaStream_t s);
cudaError_t launch_export_q_page(const KernelArgs& a, int unit, int page, uint8_t* k_codes, void* k_params,
                                 uint8_t* v_codes, void* v_params, cudaStream_t s);
cudaError_t launch_export_mass(const KernelArgs& a, int unit, float* mass, cudaStream_t s);

// dynamic shared memory the route kernel needs for a given sort capacity (power of two)
size_t route_smem_bytes(const Geometry& g, int sort_capacity);
cudaError_t route_prepare(size_t max_smem);

}  // namespace qevict
