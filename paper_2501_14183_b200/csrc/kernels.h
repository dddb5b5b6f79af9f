// Internal launch interface between the C-ABI layer and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/vardrop.h"

namespace vardrop {

// Kernel identities for the launch counter and the optional per-kernel event timer (vardrop_profile_*).
enum KernelId {
    K_HASH = 0, K_SELECT_SMALL, K_SELECT_COUNT, K_SELECT_GROUP, K_SELECT_SAMPLE, K_GATHER, K_ATTN_FWD, K_BWD_PREP, K_ATTN_BWD, K_BWD_CONVERT, K_PEARSON_NORM, K_PEARSON_MAX, K_GATHER_ROWS, K_COUNT
};
// Wrap a kernel launch: counts it and, when the timer is armed, brackets it with a pair of CUDA events on `stream`.
struct LaunchScope {
    LaunchScope(int id, cudaStream_t stream);
    ~LaunchScope();
    int id_;
    cudaStream_t stream_;
    void* stop_;
};

// hash.cu
size_t hash_workspace_bytes(const vardrop_hash_cfg& cfg);
int hash_validate(const vardrop_hash_cfg& cfg, int* f_lo, int* f_hi);
int hash_launch(const float* x, const vardrop_hash_cfg& cfg, uint64_t* keys, int32_t* freqs, float* amp_dbg, int* status,
                cudaStream_t stream);

// hash_rows.cu: register-blocked plans for selected lookback lengths; -1 = no plan for this configuration
int hash_rows_launch(const float* x, const vardrop_hash_cfg& cfg, int f_lo, int f_hi, uint64_t* keys, int32_t* freqs, float* amp_dbg,
                     int* status, cudaStream_t stream);
int sm_count();       // multiprocessors of the current device

// select.cu
size_t select_workspace_bytes(const vardrop_select_cfg& cfg);
int select_validate(const vardrop_select_cfg& cfg);
int select_launch(const uint64_t* keys, const vardrop_select_cfg& cfg, int32_t* group_id, int32_t* group_offsets, int32_t* members,
                  int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, void* ws, cudaStream_t stream);

// allocation-free variant: scratch is a fixed array inside the module
constexpr int kStaticMaxRows = 16384;                 // largest S * N it accepts
constexpr int kStaticSelectBytes = 400 * 1024;        // size of that array
int select_static_launch(const uint64_t* keys, const vardrop_select_cfg& cfg, int32_t* group_id, int32_t* group_offsets,
                         int32_t* members, int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, cudaStream_t stream);

// gather_rows.cu
int gather_rows_validate(const vardrop_gather_cfg& cfg);
int gather_rows_launch(const float* x, const int32_t* sel_idx, const int32_t* n_sel, const vardrop_gather_cfg& cfg, float* x_sel, cudaStream_t stream);

// pearson.cu
size_t pearson_workspace_bytes(const vardrop_pearson_cfg& cfg);
int pearson_validate(const vardrop_pearson_cfg& cfg);
int pearson_launch(const float* x, const vardrop_pearson_cfg& cfg, float* max_rho, int32_t* n_above, void* ws, cudaStream_t stream);

// attn_*.cu
size_t attn_workspace_bytes(const vardrop_attn_cfg& cfg);
int attn_validate(const vardrop_attn_cfg& cfg);
int attn_fwd_launch(const void* q, const void* k, const void* v, const int32_t* sel_idx, const int32_t* n_sel,
                    const vardrop_attn_cfg& cfg, void* o, float* lse, void* ws, cudaStream_t stream);
int attn_bwd_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                    const int32_t* sel_idx, const int32_t* n_sel, const int32_t* inv_idx, const vardrop_attn_cfg& cfg, void* dq,
                    void* dk, void* dv, void* ws, cudaStream_t stream);

}  // namespace vardrop
