/*
 * moe_b200.h -- C ABI of libmoe_b200.so: the MoE expert FFN, forward and backward, on one
 * NVIDIA B200 (sm_100a).
 *
 * The layer, for T tokens of width H routed to K of E experts with intermediate width I:
 *
 *   route-permute            stable sort of the (token, slot) pairs by expert into a packed,
 *                            expert-ordered row buffer with per-expert offsets
 *   grouped GEMM gate/up     per expert g = Xp.Wg[e], u = Xp.Wu[e]; Hact = silu(g) * u
 *   grouped GEMM down        per expert Yp = Hact.Wd[e]
 *   unpermute-combine        Y[t] = sum_k w[t,k] * Yp[row(t,k)]
 *
 * and the matching backward calls (dgrad and wgrad grouped GEMMs).  The packed-by-expert row
 * buffer with cumulative row counts is the layout the paper describes in its appendix on the
 * dW1 weight-gradient kernel ("What the kernel computes"); `offsets[1..E]` is that appendix's
 * inclusive cumulative-sum vector.  The weight gradient of the first projection,
 * dW1_e = X_e^T G_e over a ragged number of rows per expert, is the kernel of the paper's section
 * "Production Validation: VeOmni MoE".
 *
 * Where the calls come from: the paper covers the packed layout and one kernel, the weight gradient of the first
 * projection (moe_grouped_gemm_gateup_wgrad).  The other calls -- route-permute, the two forward GEMMs, combine, and
 * every other backward call -- are the standard expert-FFN algebra and its chain rule as this library's task
 * statement lists them; the paper is silent on them, so their comments below state the operation itself.
 *
 * Conventions for every call
 *   - Notation: R = T*K routed rows; pair id p = t*K + k (token-major).
 *   - All tensors are row-major with the last index contiguous.  `void*` tensors hold bf16
 *     (bfloat16 as 16-bit words); all results are rounded once, to nearest even, from fp32.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer to memory owned by the
 *     caller, 16-byte aligned.  The library allocates no memory, keeps no pointer after a call
 *     returns, and never synchronises: all work is enqueued on `stream` (a cudaStream_t) in
 *     order.  (One exception to "creates nothing": moe_layer_fwd_bwd_host creates two copy streams and a few
 *     events per device on its first call; see there.)  Outputs are overwritten.  Inputs and outputs must not
 *     overlap.  Nothing a call does depends
 *     on data that must first travel to the host, so a sequence of calls can be captured in a CUDA
 *     graph and replayed; run each kind of call once on the device before capturing (the first call of a
 *     kernel sets its launch attributes and queries occupancy).
 *   - H and I must be multiples of 64; 1 <= K <= E <= 1024; K <= 32; T*K < 2^31.
 *   - Return value: MOE_OK or an error code.  Argument errors are detected on the host before
 *     anything is launched.  Problems only the device can see are recorded in a per-device status word
 *     that moe_device_status() reads and clears: a kernel that gives up waiting (every device-side wait is
 *     bounded; there is never a trap) records MOE_ERR_TIMEOUT, and moe_permute records MOE_ERR_BAD_INDEX
 *     when it meets an expert id outside [0, E).
 *   - `offsets` passed to a GEMM call must be the array moe_permute produced (non-decreasing,
 *     offsets[0] = 0, offsets[E] = R).  Expert ids in topk_idx must lie in [0, E); a pair that violates this
 *     is dropped (it gets no row, offsets[E] < R then) and reported as above.
 */
#ifndef MOE_B200_H
#define MOE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t T; /* tokens */
    int32_t H; /* hidden width */
    int32_t I; /* per-expert intermediate width */
    int32_t E; /* experts */
    int32_t K; /* experts per token (top-k) */
} moe_dims_t;

typedef enum {
    MOE_OK = 0,
    MOE_ERR_NULL = 1,              /* a required pointer is NULL */
    MOE_ERR_DIMS = 2,              /* non-positive size, K > E, R overflow */
    MOE_ERR_UNSUPPORTED_SHAPE = 3, /* H or I not a multiple of 64, E or K above the limits */
    MOE_ERR_ALIGNMENT = 4,         /* a pointer is not 16-byte aligned */
    MOE_ERR_WORKSPACE = 5,         /* workspace / arena too small */
    MOE_ERR_CUDA = 6,              /* a CUDA runtime or driver call failed */
    MOE_ERR_BAD_INDEX = 7,         /* device status only: moe_permute met an expert id outside [0, E) */
    MOE_ERR_TIMEOUT = 8            /* device status only: a bounded wait inside a kernel ran out */
} moe_status_t;

typedef void* moe_stream_t; /* a cudaStream_t */

/* Human-readable name of a status code (host; never NULL). */
const char* moe_status_string(int status);

/* Bytes of device workspace moe_permute needs for these sizes (host; 0 on invalid dims). */
size_t moe_permute_workspace_bytes(const moe_dims_t* dims);

/* Reads the device status word of the current device into *status_out (host pointer) and clears
 * it.  Synchronises the device.  Returns MOE_OK or MOE_ERR_CUDA. */
int moe_device_status(int* status_out);

/* ---- a1: route-permute ----------------------------------------------------------------------
 * counts[e]      number of pairs with topk_idx = e                               int32 [E]
 * offsets        exclusive prefix of counts, offsets[E] = R                      int32 [E+1]
 * row_to_pair    pair ids sorted by (expert, pair id): a stable sort by expert   int32 [R]
 * pair_to_row    inverse of row_to_pair                                          int32 [R]
 * x_perm[r,:]  = x[row_to_pair[r] / K, :]                                        bf16  [R,H]
 * x [T,H] bf16, topk_idx [T,K] int32.  workspace: moe_permute_workspace_bytes(dims) bytes,
 * contents undefined before and after.  x_perm may be NULL (indices only).
 * Layout follows the paper's packed-by-expert buffer (appendix, "What the kernel computes").
 * A pair whose expert id is outside [0, E) is left out: it gets no row, its pair_to_row entry and the
 * rows from offsets[E] on are not written, and the device status word reads MOE_ERR_BAD_INDEX. */
int moe_permute(const moe_dims_t* dims, const void* x, const int32_t* topk_idx, void* x_perm,
                int32_t* counts, int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row,
                void* workspace, size_t workspace_bytes, moe_stream_t stream);

/* ---- route-permute for callers that cannot allocate device memory ----------------------------
 * (The paper has no counterpart of this call; it exists for integration reasons only.)
 * Same inputs, outputs and results as moe_permute, but without the workspace argument: the
 * scratch table sits in a fixed array inside the library image, MOE_PERMUTE_STATIC_SCRATCH_BYTES
 * large, which every GPU that loads the library holds until the process exits.  It is meant for
 * code that runs where a device allocation is not possible or not allowed: inside a serving or
 * training loop whose memory was handed out once at start-up and is owned by someone else's pool,
 * in a plug-in that only receives the tensors it must fill, or on a latency-critical path where
 * cudaMalloc's implicit device synchronisation is unacceptable.  The call itself makes no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Limit: returns MOE_ERR_WORKSPACE (nothing launched) when
 *     moe_permute_workspace_bytes(dims) > MOE_PERMUTE_STATIC_SCRATCH_BYTES, i.e. when
 *     ceil(T*K/256) * E * 4 bytes exceeds 4 MiB (all five benchmark configurations need <= 256 KiB).
 *   - The first call on each device looks up the array's device address (a one-time set-up on the
 *     host, with that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Its contents carry over from call to call, which
 *     is harmless here because each call overwrites every entry before reading it; but two calls
 *     whose kernels may overlap on the GPU (different streams without ordering, or different host
 *     threads) race on it and give wrong indices.  Serialise them, or use moe_permute with
 *     separate workspaces. */
#define MOE_PERMUTE_STATIC_SCRATCH_BYTES (4u << 20)
int moe_permute_static_scratch(const moe_dims_t* dims, const void* x, const int32_t* topk_idx,
                               void* x_perm, int32_t* counts, int32_t* offsets,
                               int32_t* row_to_pair, int32_t* pair_to_row, moe_stream_t stream);

/* ---- a8: dx[t,:] = sum_k dx_perm[pair_to_row[t*K+k], :]   (fp32 sum in slot order) ----------
 * The gradient of a1's row copy (chain rule; the paper has no counterpart). */
int moe_permute_bwd(const moe_dims_t* dims, const void* dx_perm, const int32_t* pair_to_row,
                    void* dx, moe_stream_t stream);

/* ---- a2: grouped GEMM gate/up with fused SwiGLU ---------------------------------------------
 * For rows r in [offsets[e], offsets[e+1]):  g = x_perm[r,:] . w_gate[e],  u = x_perm[r,:] . w_up[e]
 * (bf16 operands, fp32 accumulation);  h_act[r,:] = g / (1 + exp(-g)) * u  from the fp32 values;
 * gu_saved[r,:] = [g | u] rounded to bf16 (gate in columns [0,I), up in [I,2I)); may be NULL.
 * x_perm [R,H], w_gate, w_up [E,H,I], h_act [R,I], gu_saved [R,2I].  The gate and up
 * projections form one GEMM of width 2I as in the paper's gate_up_proj. */
int moe_grouped_gemm_gateup_swiglu(const moe_dims_t* dims, const void* x_perm, const void* w_gate,
                                   const void* w_up, const int32_t* offsets, void* h_act,
                                   void* gu_saved, moe_stream_t stream);

/* ---- a3: y_perm[r,:] = h_act[r,:] . w_down[e]      w_down [E,I,H], y_perm [R,H] --------------
 * The expert's second projection (standard expert-FFN algebra; the paper has no counterpart). */
int moe_grouped_gemm_down(const moe_dims_t* dims, const void* h_act, const void* w_down,
                          const int32_t* offsets, void* y_perm, moe_stream_t stream);

/* ---- a4: y[t,:] = sum_k topk_w[t,k] * y_perm[pair_to_row[t*K+k], :] -------------------------
 * topk_w [T,K] fp32; fp32 sum in slot order, one rounding.  y [T,H].  The routing weights enter the layer
 * here and nowhere else (standard top-k combine; the paper has no counterpart). */
int moe_unpermute_combine(const moe_dims_t* dims, const void* y_perm, const float* topk_w,
                          const int32_t* pair_to_row, void* y, moe_stream_t stream);

/* ---- a5: dy_perm[pair_to_row[p],:] = topk_w[p] * dy[t(p),:];
 *          dtopk_w[t,k] = <dy[t,:], y_perm[pair_to_row[t*K+k],:]>   (fp32 [T,K]; may be NULL,
 *          and then y_perm may be NULL too).  The chain rule applied to a4 (the paper has no counterpart). */
int moe_unpermute_combine_bwd(const moe_dims_t* dims, const void* dy, const void* y_perm,
                              const float* topk_w, const int32_t* pair_to_row, void* dy_perm,
                              float* dtopk_w, moe_stream_t stream);

/* ---- a6: down projection backward ------------------------------------------------------------
 * dgrad  dh_act[r,:] = dy_perm[r,:] . w_down[e]^T                      dh_act [R,I]
 * wgrad  dw_down[e]  = sum over rows r of expert e of h_act[r,:]^T dy_perm[r,:]   [E,I,H]
 *        (all zeros for an expert without rows; written for every expert).
 * moe_grouped_gemm_down_bwd runs the dgrad then the wgrad.  The chain rule applied to a3; the weight gradient has
 * the shape of the paper's kernel (contraction over the expert's ragged rows), the paper itself treats only a7's. */
int moe_grouped_gemm_down_dgrad(const moe_dims_t* dims, const void* dy_perm, const void* w_down,
                                const int32_t* offsets, void* dh_act, moe_stream_t stream);
int moe_grouped_gemm_down_wgrad(const moe_dims_t* dims, const void* h_act, const void* dy_perm,
                                const int32_t* offsets, void* dw_down, moe_stream_t stream);
int moe_grouped_gemm_down_bwd(const moe_dims_t* dims, const void* dy_perm, const void* h_act,
                              const void* w_down, const int32_t* offsets, void* dh_act,
                              void* dw_down, moe_stream_t stream);

/* ---- a7: SwiGLU backward and gate/up projection backward ------------------------------------
 * moe_swiglu_bwd   with s = 1/(1+exp(-g)):  dg = dh_act*u*s*(1+g*(1-s)),  du = dh_act*g*s;
 *                  dgu [R,2I] = [dg | du] (bf16), g,u read from gu_saved.
 * dgrad            dx_perm[r,:] = dg[r,:] . w_gate[e]^T + du[r,:] . w_up[e]^T          [R,H]
 * wgrad            dw_gate[e] = sum_r x_perm[r,:]^T dg[r,:],  dw_up[e] likewise         [E,H,I]
 *                  -- the paper's dW1_e = X_e^T G_e with the ragged contraction over the
 *                  expert's rows; zeros for an expert without rows.
 * moe_grouped_gemm_gateup_swiglu_bwd runs the three in this order; dgu is caller-provided
 * scratch that also returns dGU. */
int moe_swiglu_bwd(const moe_dims_t* dims, const void* dh_act, const void* gu_saved, void* dgu,
                   moe_stream_t stream);
/* Fused form of the down dgrad and moe_swiglu_bwd (an additional entry point; the two-call form stays):
 * dgu[r,:] = [dg | du] computed from dh = dy_perm[r,:] . w_down[e]^T held in fp32 -- dh_act is never
 * written, and the chain to dx loses one bf16 rounding -- and from g, u read from gu_saved [R,2I].
 * dy_perm [R,H], w_down [E,I,H], dgu [R,2I].  Replaces moe_grouped_gemm_down_dgrad + moe_swiglu_bwd. */
int moe_grouped_gemm_down_dgrad_swiglu_bwd(const moe_dims_t* dims, const void* dy_perm,
                                           const void* w_down, const void* gu_saved,
                                           const int32_t* offsets, void* dgu, moe_stream_t stream);
int moe_grouped_gemm_gateup_dgrad(const moe_dims_t* dims, const void* dgu, const void* w_gate,
                                  const void* w_up, const int32_t* offsets, void* dx_perm,
                                  moe_stream_t stream);
int moe_grouped_gemm_gateup_wgrad(const moe_dims_t* dims, const void* x_perm, const void* dgu,
                                  const int32_t* offsets, void* dw_gate, void* dw_up,
                                  moe_stream_t stream);
int moe_grouped_gemm_gateup_swiglu_bwd(const moe_dims_t* dims, const void* dh_act,
                                       const void* gu_saved, const void* x_perm,
                                       const void* w_gate, const void* w_up,
                                       const int32_t* offsets, void* dgu, void* dx_perm,
                                       void* dw_gate, void* dw_up, moe_stream_t stream);

/* ---- router in front of a1 ---------------------------------------------------------------------
 * The step that produces a1's routing inputs; the benchmark workloads describe it as "softmax
 * over router logits, top-k renormalised" (the paper itself has no counterpart: its kernel starts
 * from the packed buffer).  Uses dims->T, E, K only (1 <= K <= E <= 1024, K <= 32, T >= 1; H and I are not looked at).
 * moe_router_topk      logits [T,E] fp32 (device, no NaN).  Per token the K largest logits, slots in
 *                      descending order, equal values ordered by lower expert id, decided on the
 *                      fp32 values as given -> topk_idx [T,K] int32.  topk_w [T,K] fp32 =
 *                      exp(z_k) / sum over the kept j of exp(z_j), i.e. softmax(z) renormalised over
 *                      the kept experts (fp32 arithmetic, row maximum subtracted).
 * moe_router_topk_bwd  selection frozen: dlogits[t, topk_idx[t,k]] = w_k (dw_k - sum_j w_j dw_j),
 *                      zero for the other experts; dlogits [T,E] fp32 is written in full.
 * All pointers device, 16-byte aligned, caller-owned; status codes as everywhere else. */
int moe_router_topk(const moe_dims_t* dims, const float* logits, int32_t* topk_idx, float* topk_w,
                    moe_stream_t stream);
int moe_router_topk_bwd(const moe_dims_t* dims, const int32_t* topk_idx, const float* topk_w,
                        const float* dtopk_w, float* dlogits, moe_stream_t stream);

/* ---- block-scaled FP8 (MXFP8) twins of the six grouped GEMMs ------------------------------------
 * Lower-precision forms of the grouped GEMMs on the block-scaled tensor-core path (the paper only names FP8
 * tensor-core paths among its micro-profiling tools; the format is the OCP Microscaling MXFP8 one).  Every call works
 * on caller-owned code and scale buffers; outputs stay bf16, accumulation fp32.  First the down projection: both operands
 * as FP8 E4M3 codes with one E8M0 scale byte s (value 2^(s-127)) per 32 consecutive elements ALONG THE CONTRACTION
 * (I).  Scale of a block with largest magnitude a > 0: 2^(floor(log2 a) - 8), clamped to the E8M0 range; elements:
 * value / scale rounded to nearest even onto the E4M3 grid, magnitudes above 448 saturating; an all-zero block has
 * s = 0 and zero codes.  Products of the dequantised operands accumulate in fp32; y_perm is bf16.  The result is
 * that of the quantised operands, NOT within the bf16 tolerances of the unquantised layer (a 3-bit mantissa: a few
 * per cent relative error per tensor).  Requires H and I to be multiples of 128 (MOE_ERR_UNSUPPORTED_SHAPE otherwise).
 *   moe_mxfp8_quantize_h_act   h_act [R,I] bf16 -> codes [R,I] bytes; scales: moe_mxfp8_act_scale_bytes(dims) bytes
 *                              laid out [I/128][R][4]: the scale bytes of the 4 blocks of 32 inside the 128-wide
 *                              slice kt of row r are bytes scales[(kt*R + r)*4 + 0..3].
 *   moe_mxfp8_quantize_w_down  w_down [E,I,H] bf16 -> codes_t [E,H,I] bytes (transposed: contraction contiguous);
 *                              scales: moe_mxfp8_w_down_scale_bytes(dims) bytes holding every scale twice, once
 *                              per tiling of the two GEMM kernels (128-feature tiles on one CTA; 208-feature tiles
 *                              on a CTA pair, used from 256 rows per expert on average):
 *                              first [E][H/128][I/128][512]: the scale of feature h, block b of 32 along I, is
 *                              byte (h%32)*16 + ((h%128)/32)*4 + b%4 of the 512-byte group (e, h/128, b/4);
 *                              then [E][ceil(H/208)][I/128][1024]: with h' = h%208 the same scale is byte
 *                              (h'/128)*512 + (h'%32)*16 + ((h'%128)/32)*4 + b%4 of the 1024-byte group
 *                              (e, h/208, b/4); bytes of a group that no feature owns are left unwritten.
 *   moe_grouped_gemm_down_mxfp8  y_perm[r,:] = dequant(h row r) . dequant(w_down[e]) for rows r of expert e.
 * All pointers device, 16-byte aligned; codes and scales are caller-owned buffers. */
size_t moe_mxfp8_act_scale_bytes(const moe_dims_t* dims);
size_t moe_mxfp8_w_down_scale_bytes(const moe_dims_t* dims);
int moe_mxfp8_quantize_h_act(const moe_dims_t* dims, const void* h_act, void* codes, void* scales,
                             moe_stream_t stream);
int moe_mxfp8_quantize_w_down(const moe_dims_t* dims, const void* w_down, void* codes_t, void* scales,
                              moe_stream_t stream);
int moe_grouped_gemm_down_mxfp8(const moe_dims_t* dims, const void* h_codes, const void* h_scales,
                                const void* w_codes_t, const void* w_scales, const int32_t* offsets,
                                void* y_perm, moe_stream_t stream);

/* The data gradient of the down projection on the same kernels: dh_act[r,:] = dequant(dy row r) . dequant(w_down[e])^T
 * with both operands block-scaled along ITS contraction, H (defined by the benchmark spec's backward counterparts
 * and the format above; the paper has no FP8 path of its own).  w_down [E,I,H] is already contraction-contiguous:
 *   moe_mxfp8_quantize_dy_perm       dy_perm [R,H] bf16 -> codes [R,H] bytes; scales: moe_mxfp8_dy_scale_bytes(dims)
 *                                    bytes laid out [H/128][R][4] (as the activation scales above, slices along H).
 *   moe_mxfp8_quantize_w_down_dgrad  w_down [E,I,H] bf16 -> codes [E,I,H] bytes (same layout); scales:
 *                                    moe_mxfp8_w_down_dgrad_scale_bytes(dims) bytes, the two tilings described above
 *                                    with the roles of the axes exchanged (feature = i, 128-wide slices along H).
 *   moe_grouped_gemm_down_dgrad_mxfp8  dh_act [R,I] bf16, overwritten.
 * Same requirements, status codes and tolerance statement as the forward call. */
size_t moe_mxfp8_dy_scale_bytes(const moe_dims_t* dims);
size_t moe_mxfp8_w_down_dgrad_scale_bytes(const moe_dims_t* dims);
int moe_mxfp8_quantize_dy_perm(const moe_dims_t* dims, const void* dy_perm, void* codes, void* scales,
                               moe_stream_t stream);
int moe_mxfp8_quantize_w_down_dgrad(const moe_dims_t* dims, const void* w_down, void* codes, void* scales,
                                    moe_stream_t stream);
int moe_grouped_gemm_down_dgrad_mxfp8(const moe_dims_t* dims, const void* dy_codes, const void* dy_scales,
                                      const void* w_codes, const void* w_scales, const int32_t* offsets,
                                      void* dh_act, moe_stream_t stream);

/* The data gradient of the gate/up projection likewise: dx_perm[r,:] = dequant(dgu row r) . dequant([w_gate[e] |
 * w_up[e]])^T, contraction over the 2I gate and up features (blocks of 32 never straddle the boundary: I is a
 * multiple of 128).  w_gate, w_up [E,H,I] are contraction-contiguous as they lie; their codes go side by side:
 *   moe_mxfp8_quantize_dgu             dgu [R,2I] bf16 -> codes [R,2I] bytes; scales: moe_mxfp8_dgu_scale_bytes(dims)
 *                                      bytes laid out [2I/128][R][4].
 *   moe_mxfp8_quantize_w_gateup_dgrad  w_gate, w_up -> codes [E,H,2I] bytes (gate columns first); scales:
 *                                      moe_mxfp8_w_gateup_dgrad_scale_bytes(dims) bytes, the two tilings with
 *                                      feature = h and 128-wide slices along the 2I columns.
 *   moe_grouped_gemm_gateup_dgrad_mxfp8  dx_perm [R,H] bf16, overwritten.
 * Same requirements, status codes and tolerance statement as the forward call. */
size_t moe_mxfp8_dgu_scale_bytes(const moe_dims_t* dims);
size_t moe_mxfp8_w_gateup_dgrad_scale_bytes(const moe_dims_t* dims);
int moe_mxfp8_quantize_dgu(const moe_dims_t* dims, const void* dgu, void* codes, void* scales, moe_stream_t stream);
int moe_mxfp8_quantize_w_gateup_dgrad(const moe_dims_t* dims, const void* w_gate, const void* w_up, void* codes,
                                      void* scales, moe_stream_t stream);
int moe_grouped_gemm_gateup_dgrad_mxfp8(const moe_dims_t* dims, const void* dgu_codes, const void* dgu_scales,
                                        const void* w_codes, const void* w_scales, const int32_t* offsets,
                                        void* dx_perm, moe_stream_t stream);
/* moe_swiglu_bwd with the quantiser of its result fused in: dgu exactly as moe_swiglu_bwd writes it, and dgu_codes /
 * dgu_scales = what moe_mxfp8_quantize_dgu makes of that dgu (one pass over the data instead of two). */
int moe_swiglu_bwd_mxfp8(const moe_dims_t* dims, const void* dh_act, const void* gu_saved, void* dgu, void* dgu_codes,
                         void* dgu_scales, moe_stream_t stream);

/* The gate/up projection itself: gu[r,:] = [ dequant(x row r) . dequant(w_gate[e]) | dequant(x row r) . dequant(w_up[e]) ],
 * contraction over H; every gate / up feature has its own scales along H.  The SwiGLU activation is a second call that
 * also emits the block-scaled FP8 form of its result, so that the FP8 down projection needs no separate quantiser:
 *   moe_mxfp8_quantize_x_perm    x_perm [R,H] bf16 -> codes [R,H] bytes; scales: moe_mxfp8_x_scale_bytes(dims) bytes,
 *                                [H/128][R][4].
 *   moe_mxfp8_quantize_w_gateup  w_gate, w_up [E,H,I] -> codes_t [E,2I,H] bytes (transposed: contraction contiguous;
 *                                gate features first); scales: moe_mxfp8_w_gateup_scale_bytes(dims) bytes, the two
 *                                tilings with feature = gate/up column and 128-wide slices along H.
 *   moe_grouped_gemm_gateup_mxfp8  gu [R,2I] bf16 (gate columns [0,I), up columns [I,2I)), overwritten.
 *   moe_swiglu_mxfp8             gu [R,2I] bf16 -> h_act [R,I] bf16 = silu(g)*u (fp32, rounded once), and h_codes /
 *                                h_scales = the quantised form of exactly those bf16 values, laid out as
 *                                moe_mxfp8_quantize_h_act writes them.  Elementwise, HBM-bound.
 * Same requirements, status codes and tolerance statement as the other block-scaled calls. */
size_t moe_mxfp8_x_scale_bytes(const moe_dims_t* dims);
size_t moe_mxfp8_w_gateup_scale_bytes(const moe_dims_t* dims);
int moe_mxfp8_quantize_x_perm(const moe_dims_t* dims, const void* x_perm, void* codes, void* scales, moe_stream_t stream);
int moe_mxfp8_quantize_w_gateup(const moe_dims_t* dims, const void* w_gate, const void* w_up, void* codes_t, void* scales,
                                moe_stream_t stream);
int moe_grouped_gemm_gateup_mxfp8(const moe_dims_t* dims, const void* x_codes, const void* x_scales,
                                  const void* w_codes_t, const void* w_scales, const int32_t* offsets, void* gu,
                                  moe_stream_t stream);
int moe_swiglu_mxfp8(const moe_dims_t* dims, const void* gu, void* h_act, void* h_codes, void* h_scales,
                     moe_stream_t stream);

/* The two weight gradients, whose contraction runs over the packed rows of each expert (the paper's dW1 kernel is the
 * bf16 form of the second; its section "Production Validation: VeOmni MoE" defines dW1_e = X_e^T G_e): both operands are
 * quantised along the TOKEN axis, every column in blocks of 32 consecutive rows counted from the expert's first row (a
 * block never holds rows of two experts; an expert's last block may be short), and stored transposed and padded:
 *   moe_mxfp8_quantize_tokens  columns [col0, col0 + n_features) of x [R, ld] bf16 (ld, col0 multiples of 8; n_features a
 *                              multiple of 128) -> codes_t [n_features, P] bytes with P = roundup(R,128) + 128*E:
 *                              column slice_prefix[e]*128 + i holds row offsets[e] + i, each expert's columns padded with
 *                              zero codes to a multiple of 128 (columns after the last expert's are not written);
 *                              scales (moe_mxfp8_tokens_scale_bytes): slice_prefix[E+1] as int32 in the first 8192
 *                              bytes, then the scale bytes as [P/128][n_features][4], then again tiled per 208 features
 *                              [ceil(n/208)][P/128][1024] for use as the N-side operand.  Two launches.
 *   moe_grouped_gemm_down_wgrad_mxfp8    dw_down [E,I,H] bf16 = Q(h_act)^T Q(dy_perm) per expert, from the token-
 *                              quantised h_act (n_features = I) and dy_perm (n_features = H).
 *   moe_grouped_gemm_gateup_wgrad_mxfp8  dw_gate, dw_up [E,H,I] bf16 from the token-quantised x_perm (n_features = H)
 *                              and the two halves of dgu quantised separately (col0 = 0 and col0 = I, n_features = I,
 *                              ld = 2I).  Two launches.
 * Every expert's gradient is written, zeros for an expert without rows.  The row counts come from the slice_prefix in
 * the first operand's scales (the offsets the quantiser was given).  Same requirements, status codes and tolerance
 * statement as the other block-scaled calls. */
size_t moe_mxfp8_tokens_codes_bytes(const moe_dims_t* dims, int n_features);
size_t moe_mxfp8_tokens_scale_bytes(const moe_dims_t* dims, int n_features);
int moe_mxfp8_quantize_tokens(const moe_dims_t* dims, const void* x, int ld, int col0, int n_features,
                              const int32_t* offsets, void* codes_t, void* scales, moe_stream_t stream);
int moe_grouped_gemm_down_wgrad_mxfp8(const moe_dims_t* dims, const void* h_codes_t, const void* h_scales,
                                      const void* dy_codes_t, const void* dy_scales, void* dw_down,
                                      moe_stream_t stream);
int moe_grouped_gemm_gateup_wgrad_mxfp8(const moe_dims_t* dims, const void* x_codes_t, const void* x_scales,
                                        const void* dg_codes_t, const void* dg_scales, const void* du_codes_t,
                                        const void* du_scales, void* dw_gate, void* dw_up, moe_stream_t stream);

/* ---- whole layer from HOST activations ------------------------------------------------------
 * One training step of the layer for a caller whose per-step tensors live in host memory:
 * copies x, topk_idx, topk_w, dy (HOST pointers; pinned memory makes the copies asynchronous)
 * into the device arena, runs a1..a8, and copies y [T,H], dx [T,H] (bf16) and dtopk_w [T,K]
 * (fp32) back to HOST pointers.  Weights w_* and weight gradients dw_* are DEVICE pointers (the
 * parameters stay resident, as in training).  `arena` is device scratch of at least
 * moe_layer_arena_bytes(dims) bytes holding every intermediate of the step.  The kernels are
 * enqueued on `stream`; the uploads and the downloads run on two internal copy streams per
 * device (created on the first call, the only CUDA objects the library ever creates), tied to
 * `stream` with events: y comes down under the backward pass, dx and dtopk_w under the two
 * weight-gradient GEMMs (which run last: nothing downstream waits for them), and the uploads of a
 * call start as soon as the PREVIOUS call's last reader of the arena's input blocks is done, so
 * that back-to-back calls overlap the next step's uploads with this step's backward GEMMs.
 * Consequences for the caller: (1) the host results are valid after `stream` is synchronised;
 * (2) the host INPUT buffers are read from the moment of the call on, not in stream order: they
 * must hold their final values when the function is called and stay untouched until `stream`
 * has passed this call; (3) successive calls that share an arena must be made on the same stream,
 * and nothing else may write to the arena between them (the uploads of a call do not wait for
 * other work on `stream`);
 * (4) the first call on a device orders its uploads after all work already on `stream`.
 * Not safe to call from two host threads at once on the same device. */
size_t moe_layer_arena_bytes(const moe_dims_t* dims);
int moe_layer_fwd_bwd_host(const moe_dims_t* dims, const void* x_host, const int32_t* topk_idx_host,
                           const float* topk_w_host, const void* dy_host, const void* w_gate,
                           const void* w_up, const void* w_down, void* y_host, void* dx_host,
                           float* dtopk_w_host, void* dw_gate, void* dw_up, void* dw_down,
                           void* arena, size_t arena_bytes, moe_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H */
