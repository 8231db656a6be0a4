// Host-side launchers of the libadsa kernels (one per kernel family).
#pragma once

#include <cuda.h>
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

// The staged cluster kernel (attention alone, or the whole layer-step fused).
constexpr int kStepMaxGroups = 64;             // copy groups (mbarriers) per CTA
constexpr int kStepSmemLimit = 200 * 1024;     // dynamic shared memory a CTA may ask for

struct StepPlan {
    int cluster_size;   // CTAs per stream (1, 2, 4 or 8); 0 = the stream does not fit, use the streaming kernels
    int chunk_rows;     // rows per CTA
    int group_rows;     // rows per copy group
    size_t smem_bytes;
};
StepPlan plan_step(const DevCtx &c, int n_rows, bool fused, int sm_count, int chunk_target);
cudaError_t launch_step(const DevCtx &c, const StepPlan &plan, bool fused, int layer, int cur_pos, int budget_rows,
                        const void *q, const void *k_new, const void *v_new, void *out_bf16, float *out_f32,
                        cudaStream_t st);
cudaError_t configure_step_kernel(const DevCtx &c);
cudaError_t launch_scores_copy(const DevCtx &c, int layer, int cur_pos, float *scores_out, cudaStream_t st);

// The persistent pipelined kernel (attention alone, or the whole layer-step fused).
constexpr int kPMaxStages = 24;                // ring stages (a K tile + a V tile each)
constexpr int kPSmemLimit = 220 * 1024;        // dynamic shared memory of the one CTA per SM

struct PStepPlan {
    int n_stages;       // 0 = the configuration does not fit
    int grid;           // CTAs (at most one per SM)
    int tile_rows;
    size_t smem_bytes;
};
PStepPlan plan_pstep(const DevCtx &c, bool fused, int sm_count, int max_stages);
cudaError_t launch_pstep(const DevCtx &c, const PStepPlan &plan, bool fused, int layer, int cur_pos, int budget_rows,
                         const void *q, const void *k_new, const void *v_new, void *out_bf16, float *out_f32,
                         cudaStream_t st);
cudaError_t configure_pstep_kernel(const DevCtx &c);

// The warp-per-stream kernel with tensor-core arithmetic (pools with 64-element rows).
struct WStepMaps {
    CUtensorMap k[6], v[6];   // boxes of 1, 2, 4, 8, 16, 32 rows x 64 elements, 128-byte swizzle
};
constexpr int kWSmemLimit = 226 * 1024;        // dynamic shared memory of the one CTA per SM
struct WStepPlan {
    int n_groups;       // streams a CTA serves at a time; 0 = not supported / does not fit
    int group_warps;    // warps that share a stream
    int depth;          // tiles in flight per warp
    int l2_ahead;       // tiles asked into L2 beyond those in flight
    int grid;
    size_t smem_bytes;
};
bool wstep_supported(const DevCtx &c);
int build_wstep_maps(const DevCtx &c, WStepMaps *out);   // 0 on success
WStepPlan plan_wstep(const DevCtx &c, bool fused, int sm_count, int max_depth, int group_warps, int n_run = 1);
cudaError_t launch_wstep(const DevCtx &c, const WStepPlan &plan, const WStepMaps &maps, bool fused, int layer, int cur_pos,
                         int budget_rows, const void *q, const void *k_new, const void *v_new, void *out_bf16,
                         float *out_f32, cudaStream_t st, bool have_svec, bool early_state, bool use_note,
                         int next_layer, int next_tiles, int n_run = 1, const int *in_ready = nullptr, int in_epoch = 0);
cudaError_t configure_wstep_kernel(const DevCtx &c);

// Entering the condition: dense causal attention over n_rows rows per stream of a layer, and the 2-D rotary embedding.
cudaError_t launch_prefill_attn(const DevCtx &c, const void *q, const void *k, const void *v, void *out_bf16, float *out_f32,
                                int n_rows, cudaStream_t st);
cudaError_t launch_rope_2d(const DevCtx &c, void *x, const int32_t *pos, long long n_rows, float base, cudaStream_t st);

// One-time per-process kernel attribute setup (dynamic shared memory opt-in).
cudaError_t configure_kernels(const DevCtx &c);
cudaError_t configure_select_kernel(const DevCtx &c);
cudaError_t configure_score_kernel(const DevCtx &c);
cudaError_t configure_update_kernel(const DevCtx &c);

}  // namespace adsa
