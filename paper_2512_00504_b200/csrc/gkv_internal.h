// Host-side internals of the G-KV library: the context, the workspace layout and the kernel
// launchers that the C-ABI entry points call.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "gkv.h"

namespace gkv {

// Offsets (bytes) of the regions of the caller-allocated workspace.
struct WorkspaceLayout {
    uint64_t status;      // int32[64]   latched device status + diagnostics
    uint64_t seq_done;    // int32[L*batch]         CTA completion counters per (layer, sequence)
    uint64_t kept;        // int32[units_per_layer * b]   kept lists of the staged eviction path
    uint64_t fscratch;    // fp32[units_per_layer * C]    merged scores of the staged eviction path
    uint64_t prompt_sums; // fp32[units_per_layer * max_prompt]  window sums of a prompt being compressed
    uint64_t prompt_len;  // int32[batch]                        device copy of the prompt lengths
    uint64_t prompt_f;    // fp32[(1 or 2) * units_per_layer * max_prompt]  scores of long prompts (max_prompt > 8192)
    uint64_t fsel;        // fp32[units_per_layer * C]    selection scores of the staged path (redundancy term on)
    uint64_t inv_norm;    // fp32[L * units_per_layer * C] 1 / (|K row| + eps)            (redundancy term on)
    uint64_t cbar;        // fp32[L * units_per_layer * C] redundancy level of every row  (redundancy term on)
    uint64_t total;
};

struct DecodeLaunch {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* out;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    float* sacc;
    int32_t* len;        // plane 0 of the len buffer
    int32_t* seq_done;
    int32_t* status;
    int32_t* work_next;  // two zeroed words: the next item's number minus the grid size, and the CTAs that are done
    int layer0, n_layers, batch, h_q, h_kv, g, C;
    int accum;           // 1 on window steps
    int sm_count;        // SMs of the device (sizes the persistent grid)
    // filled in by decode_plan():
    int splits;          // every unit is `splits` work items, each a contiguous share of the keys; > 1: the kernel is
                         // launched in clusters of `splits` CTAs, one cluster per unit
    int stages, grid, tmem_cols;
    float scale_log2;    // log2(e) / sqrt(d)
};

// Tensor maps of the decode kernel: K and V as [rows][128] bf16 with 64-row boxes (full tiles) and with 16-row
// boxes (the ragged last tile of a unit is fetched in 16-row pieces, so at most 15 rows past the cache's end
// cross the memory bus instead of up to 63).
struct DecodeMaps {
    CUtensorMap k64, v64, k16, v16;
};

struct EvictLaunch {
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    float* f;
    float* sacc;
    int32_t* pos;        // may be NULL
    int32_t* len;        // plane 0; plane 1 (n_hist) follows at len + L_total*batch
    int32_t* seq_done;
    int32_t* kept_out;   // may be NULL: [units in launch][b]
    int32_t* kept_ws;    // staged path scratch
    float* f_ws;         // staged path scratch
    int32_t* status;
    int32_t* work;       // two zeroed words of the fused kernel: the next unit's number minus the grid size, CTAs done
    int sm_count;        // SMs of the device (sizes the fused kernel's persistent grid)
    int layer0, n_layers, L_total, batch, h_kv, C, b, w;
    float alpha;
    int mode;
    // redundancy term: selection on lambda * F - (1 - lambda) * exp(cbar - max cbar); cbar == NULL turns it off
    int32_t* evict_log;  // may be NULL: [all units][C - b] evicted positions of this step, -1 padded
    const float* cbar;   // [all units][C]
    float* fsel_ws;      // staged path scratch
    float lambda;
    int pool_kernel;     // > 1: sequence-wise max-pooling of the score before the selection
    int policy, n_sink;  // GKV_POLICY_STREAMING: the kept list is the first n_sink rows and the most recent b - n_sink
};

struct PromptLaunch {
    const __nv_bfloat16* k_src;  // [batch][h_kv][P_max][d] prefill keys / values
    const __nv_bfloat16* v_src;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    float* f;
    float* sacc;
    int32_t* pos;                // may be NULL
    int32_t* len;                // plane 0; plane 1 follows at len + L_total*batch
    const float* sums;           // [batch*h_kv][P_max] w * S of the prompt's window
    const float* cbar;           // NULL, or [batch*h_kv][P_max] redundancy level of the prompt's keys
    float lambda;                // weight of the score against the redundancy term
    float* f_long;               // NULL, or [batch*h_kv][P_max] (pooling: twice that): the scores of a prompt too long
                                 // for shared memory are kept here
    const int32_t* prompt_len;   // device [batch]
    int32_t* seq_done;
    int32_t* kept_out;           // may be NULL: [batch*h_kv][b], -1 padded
    int32_t* status;
    int layer, L_total, batch, h_kv, C, P_max, b, w, pool_kernel;
    int policy, n_sink;
};

struct RedundancyLaunch {
    const __nv_bfloat16* k_cache;
    const int32_t* len;
    float* inv_norm;     // [all units][C]
    float* cbar;         // [all units][C]
    int32_t* status;
    int layer0, n_layers, batch, h_kv, C, recent;
    float tau, eps;
};

struct ScoreLaunch {
    const __nv_bfloat16* q_win;  // [n_layers][batch][h_q][w][d]
    float* sacc;                 // receives w * S
    const int32_t* len;
    int32_t* status;
    int layer0, n_layers, batch, h_q, h_kv, g, C, w;
    int sm_count;                // SMs of the device (sizes the tensor-core kernel's persistent grid)
    float scale_log2;
};

}  // namespace gkv

struct gkv_ctx {
    gkv_config cfg;
    gkv_buffers buf;
    gkv::WorkspaceLayout ws;
    int C, g, units_per_layer;
    int device, sm_count;
    CUtensorMap tm_k, tm_v;   // 64-row boxes
    CUtensorMap tm_k16, tm_v16;   // 16-row boxes
    CUtensorMap tm_k128;          // 128-row boxes (the tensor-core scoring kernel's key tiles)
    std::vector<int32_t> len, n_hist, since_evict, sacc_valid, stage_next, cbar_valid;
    int64_t launches;
    int32_t* evict_log;  // caller's device buffer for the eviction log, or NULL
    gkv_sizes sizes;
};

namespace gkv {

int decode_pick_splits(int units_in_launch, int C, int sm_count);
void decode_plan(DecodeLaunch* p, int max_pieces);
void decode_plan_resources(const DecodeLaunch& p, int* ctas_per_sm, size_t* smem_bytes);   // of a planned launch
cudaError_t launch_decode(const DecodeLaunch& p, const DecodeMaps& maps, cudaStream_t s);
cudaError_t launch_evict_fused(const EvictLaunch& p, cudaStream_t s);
void evict_plan(const EvictLaunch& p, int* stages, int* grid, size_t* smem, int* ctas_per_sm);   // shape of that launch
cudaError_t launch_evict_merge(const EvictLaunch& p, cudaStream_t s);
cudaError_t launch_evict_select(const EvictLaunch& p, cudaStream_t s);
cudaError_t launch_evict_compact(const EvictLaunch& p, int sm_count, cudaStream_t s);
cudaError_t launch_score(const ScoreLaunch& p, const CUtensorMap& tm_k, cudaStream_t s);
cudaError_t launch_score_tc(const ScoreLaunch& p, const CUtensorMap& tm_k, const CUtensorMap& tm_q, int wk, cudaStream_t s);
int score_tc_rows_per_cta(int g, int w);
struct ScoreTcPlan { int items, items_per_unit, rows, q_bufs, stages, grid; size_t smem; };
void score_tc_plan(const ScoreLaunch& p, int wk, ScoreTcPlan* out);
int score_tc_q_box_rows(int wk);
constexpr int kScoreTcKeyBoxRows = 128;   // rows of one box of the key tensor map that launch_score_tc takes
cudaError_t score_tc_kernel_setup();
cudaError_t launch_prompt_compress(const PromptLaunch& p, cudaStream_t s);
cudaError_t launch_keynorm(const RedundancyLaunch& p, cudaStream_t s);
cudaError_t launch_redundancy(const RedundancyLaunch& p, const CUtensorMap& tm_k, cudaStream_t s);
cudaError_t redundancy_kernel_setup();
cudaError_t decode_kernel_setup();
cudaError_t score_kernel_setup();

}  // namespace gkv
