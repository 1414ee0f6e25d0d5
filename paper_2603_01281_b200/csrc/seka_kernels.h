// Internal host-side launchers shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "seka_common.cuh"

namespace seka {

// Operand preparation of the fused kernel (tile flags, edited keys of the tiles with highlighted tokens; see seka_prep.cu).  With
// `sigma` set, the routing coefficients of Eq. 6 are computed inside the launch from Q_route (the caller's Q in its own
// dtype) instead of being read from `alpha`, and written to `alpha_out` if that is not null.
seka_status launch_prep_steering(const seka_shape* s, const SteerPlan& plan, const void* K16, const float* U,
                                 const float* alpha, const float* gain, const uint8_t* head_enable, const uint8_t* mask,
                                 void* X, uint8_t* tile_hot, int* first_hot, uint8_t* bh_info, int* status, int n_tiles, cudaStream_t st,
                                 const void* Q_route = nullptr, const float* sigma = nullptr, int k_route = 0,
                                 float* alpha_out = nullptr);
// `bh_info` (null: no steering) is the per-(sequence, KV head) byte the preparation launch wrote
void launch_build_items(const Sched& sc, const int* cu, const uint8_t* bh_info, ItemRecord* items, int* count,
                        cudaStream_t st);
void launch_compact_mask(const uint8_t* mask, int T, int* list, int* count, cudaStream_t st);
void launch_convert_bf16(const float* Q, void* q16, size_t nq, const float* K, void* k16, const float* V, void* v16, size_t nk,
                         cudaStream_t st);

// Preparation of the tile-wise edit: P[m][h] = U_m U_m^T (two bf16 parts), tile flags, list of the tiles that hold a
// highlighted token; with `first_hot` / `bh_info` set also what the fused forward needs (see prep_edit_kernel); with
// `sigma` set also the routing coefficients of Eq. 6 into `alpha_out` (further blocks of the same launch).
seka_status launch_prep_edit(const seka_shape* s, const float* U, const uint8_t* mask, void* P, uint8_t* tile_hot, int n_tiles,
                             int* hot_list, int* hot_count, cudaStream_t st, int* first_hot = nullptr, uint8_t* bh_info = nullptr,
                             const float* gain = nullptr, const float* alpha = nullptr, const uint8_t* head_enable = nullptr,
                             const void* Q_route = nullptr, const float* sigma = nullptr, int k_route = 0,
                             float* alpha_out = nullptr);

// Eq. 6 for every (sequence, KV head): the launch behind adaseka_route
seka_status launch_route(const seka_shape* s, const void* Q, const float* U, const float* sigma, int k_route,
                         float* alpha_out, cudaStream_t st);

// The edited keys of the tiles that hold a highlighted token into the side buffer X [T, Hkv, 2 d] of the fused forward
// (high | low parts), by the tile kernels of the stand-alone edit in their side mode (two launches with the
// preparation): the pipelined kernel for one expert, the bank kernel for several (n_experts * d <= 512).
// K16 is the bf16 key tensor; workspace regions as in workspace_layout.
seka_status launch_stage_keys_pipe(const seka_shape* s, const WorkspaceLayout& w, const void* K16, void* X,
                                   const uint8_t* mask, const float* U, const float* alpha, const float* gain,
                                   const uint8_t* head_enable, char* ws, cudaStream_t st, const void* Q_route = nullptr,
                                   const float* sigma = nullptr, int k_route = 0);

// bf16 tensor [T, H, d] viewed as (d, H, T) for TMA: tiles of 64 x 1 x box_rows with the 128-byte swizzle.
bool make_tile_map(CUtensorMap* m, const void* base, int d, int H, long long T, int box_rows = 128);

seka_status validate_shape(const seka_shape* s);

// Number of SMs of the current device (looked up once per device, thread-safe).
bool device_info(int* n_sm);

}  // namespace seka
