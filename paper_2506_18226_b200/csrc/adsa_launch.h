// Host-side launchers of the libadsa kernels (one per kernel family).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace adsa {

struct DevCtx;

struct AttnPlan {
    int n_splits;    // chunks per stream
    int chunk_rows;  // cached rows per chunk (a multiple of 32)
};

cudaError_t launch_reset(const DevCtx &c, int n_streams, cudaStream_t st);
cudaError_t launch_append_rows(const DevCtx &c, int layer, const void *k, const void *v, const int32_t *pos,
                               int n_rows, int first_pos, cudaStream_t st);
cudaError_t launch_set_rows(const DevCtx &c, int sid, const void *k, const void *v, const int32_t *pos, int n_rows,
                            cudaStream_t st);
cudaError_t launch_kv_update(const DevCtx &c, int layer, int cur_pos, const void *k_new, const void *v_new,
                             cudaStream_t st);
size_t kv_update_smem_bytes(const DevCtx &c);

cudaError_t launch_score(const DevCtx &c, int layer, int cur_pos, float *scores_out, cudaStream_t st);
cudaError_t launch_select(const DevCtx &c, int layer, int cur_pos, int budget_rows, int32_t *sel_slots,
                          int32_t *sel_pos, int32_t *evict_pos, int32_t *counts_out, cudaStream_t st);
size_t select_smem_bytes(const DevCtx &c);

cudaError_t launch_attn(const DevCtx &c, const AttnPlan &plan, int layer, int cur_pos, const void *q,
                        const void *k_new, const void *v_new, void *out_bf16, float *out_f32, cudaStream_t st);

// One-time per-process kernel attribute setup (dynamic shared memory opt-in).
cudaError_t configure_kernels(const DevCtx &c);
cudaError_t configure_select_kernel(const DevCtx &c);
cudaError_t configure_update_kernel(const DevCtx &c);

}  // namespace adsa
