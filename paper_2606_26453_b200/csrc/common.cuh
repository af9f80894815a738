// Shared declarations of the library's translation units (internal; not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moe_b200.h"

namespace moe {

typedef __nv_bfloat16 bf16;

// Device status word (one per device that loaded the library; lives in grouped_gemm.cu): kernels
// record MOE_ERR_TIMEOUT there when a bounded wait runs out.  Synchronises the device.
int read_and_clear_device_status(int* status_out);
int movement_read_and_clear_status(int* status_out);   // the data-movement kernels' word (movement.cu)
int mx_read_and_clear_status(int* status_out);         // the block-scaled FP8 kernels' word (mxfp8.cu)

// Number of SMs of the current device (cached per device ordinal).
int sm_count();

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA; }

// ---- data-movement kernels (movement.cu) ------------------------------------------------------
int launch_permute(const moe_dims_t& d, const bf16* x, const int32_t* topk_idx, bf16* x_perm,
                   int32_t* counts, int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row,
                   void* workspace, cudaStream_t s);
size_t permute_workspace_bytes(const moe_dims_t& d);
int launch_permute_static_scratch(const moe_dims_t& d, const bf16* x, const int32_t* topk_idx, bf16* x_perm,
                                  int32_t* counts, int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row,
                                  cudaStream_t s);
int launch_gather_sum(const moe_dims_t& d, const bf16* src_perm, const float* topk_w,
                      const int32_t* pair_to_row, bf16* dst, cudaStream_t s);  // topk_w may be NULL (unit weights)
int launch_combine_bwd(const moe_dims_t& d, const bf16* dy, const bf16* y_perm, const float* topk_w,
                       const int32_t* pair_to_row, bf16* dy_perm, float* dtopk_w, cudaStream_t s);
int launch_swiglu_bwd(const moe_dims_t& d, const bf16* dh_act, const bf16* gu, bf16* dgu, cudaStream_t s);

// ---- router (router.cu) ------------------------------------------------------------------------
int launch_router_topk(const moe_dims_t& d, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t s);
int launch_router_topk_bwd(const moe_dims_t& d, const int32_t* topk_idx, const float* topk_w, const float* dtopk_w,
                           float* dlogits, cudaStream_t s);

// ---- grouped GEMMs (grouped_gemm.cu) -----------------------------------------------------------
int launch_gateup_fwd(const moe_dims_t& d, const bf16* x_perm, const bf16* w_gate, const bf16* w_up,
                      const int32_t* offsets, bf16* h_act, bf16* gu, cudaStream_t s);
int launch_down_fwd(const moe_dims_t& d, const bf16* h_act, const bf16* w_down, const int32_t* offsets,
                    bf16* y_perm, cudaStream_t s);
int launch_down_dgrad(const moe_dims_t& d, const bf16* dy_perm, const bf16* w_down, const int32_t* offsets,
                      bf16* dh_act, cudaStream_t s);
int launch_down_wgrad(const moe_dims_t& d, const bf16* h_act, const bf16* dy_perm, const int32_t* offsets,
                      bf16* dw_down, cudaStream_t s);
int launch_down_dgrad_swiglu_bwd(const moe_dims_t& d, const bf16* dy_perm, const bf16* w_down, const bf16* gu,
                                 const int32_t* offsets, bf16* dgu, cudaStream_t s);
int launch_gateup_dgrad(const moe_dims_t& d, const bf16* dgu, const bf16* w_gate, const bf16* w_up,
                        const int32_t* offsets, bf16* dx_perm, cudaStream_t s);
int launch_gateup_wgrad(const moe_dims_t& d, const bf16* x_perm, const bf16* dgu, const int32_t* offsets,
                        bf16* dw_gate, bf16* dw_up, cudaStream_t s);

// ---- block-scaled FP8 down projection (mxfp8.cu) -------------------------------------------------
size_t mx_w_scale_single_bytes(int E, int n_feat, int k);   // weight scales in the single-CTA tiling
size_t mx_w_scale_bytes(int E, int n_feat, int k);          // both tilings, one after the other
int launch_mx_quantize_rows(long long rows, int n, const bf16* x, uint8_t* codes, uint8_t* scales, cudaStream_t s);
int launch_mx_quantize_w_transposed(int E, int k, int n, int n_total, int n_off, const bf16* w, uint8_t* codes_t, uint8_t* scales,
                                    cudaStream_t s);
int launch_mx_quantize_w_rows(int E, int n_feat, int k, int k_total, int k_off, const bf16* w, uint8_t* codes, uint8_t* scales,
                              cudaStream_t s);
long long mx_tokens_pitch(long long R, int E);            // columns of a token-quantised (transposed) operand
size_t mx_tokens_scale_bytes(long long R, int E, int n);
int launch_mx_quantize_tokens(long long R, int E, const bf16* x, long long ld, int col0, int n, const int32_t* offsets,
                              uint8_t* codes_t, uint8_t* scales, cudaStream_t s);
int launch_mx_wgrad(long long R, int E, int M, int N, const uint8_t* a_codes_t, const uint8_t* a_scales, const uint8_t* b_codes_t,
                    const uint8_t* b_scales, bf16* dw, cudaStream_t s);
int launch_mx_swiglu_quantize(long long rows, int I, const bf16* gu, bf16* h_act, uint8_t* codes, uint8_t* scales, cudaStream_t s);
int launch_mx_swiglu_bwd_quantize(long long rows, int I, const bf16* dh_act, const bf16* gu, bf16* dgu, uint8_t* codes,
                                  uint8_t* scales, cudaStream_t s);
int launch_mx_gemm(long long R, int E, int n_feat, int k, const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                   const uint8_t* b_scales, const int32_t* offsets, bf16* out, cudaStream_t s);

}  // namespace moe
