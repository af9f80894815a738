// C ABI of libmoe_b200.so: argument validation and dispatch to the kernels.  See include/moe_b200.h.
#include "common.cuh"

namespace moe {

int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

namespace {

int check_dims(const moe_dims_t* d) {
    if (d == nullptr) return MOE_ERR_NULL;
    if (d->T <= 0 || d->H <= 0 || d->I <= 0 || d->E <= 0 || d->K <= 0 || d->K > d->E) return MOE_ERR_DIMS;
    if ((long long)d->T * d->K >= (1ll << 31)) return MOE_ERR_DIMS;
    if (d->H % 64 != 0 || d->I % 64 != 0 || d->E > 1024 || d->K > 32) return MOE_ERR_UNSUPPORTED_SHAPE;
    return MOE_OK;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Validation helper: every pointer in `req` must be non-NULL and 16-byte aligned; pointers in `opt`
// only need alignment when present.
template <size_t NR, size_t NO>
int check_ptrs(const void* const (&req)[NR], const void* const (&opt)[NO]) {
    for (size_t i = 0; i < NR; ++i) {
        if (req[i] == nullptr) return MOE_ERR_NULL;
        if (misaligned(req[i])) return MOE_ERR_ALIGNMENT;
    }
    for (size_t i = 0; i < NO; ++i)
        if (opt[i] != nullptr && misaligned(opt[i])) return MOE_ERR_ALIGNMENT;
    return MOE_OK;
}

#define MOE_VALIDATE(dims, ...)                                \
    do {                                                       \
        int st_ = check_dims(dims);                            \
        if (st_ != MOE_OK) return st_;                         \
        st_ = check_ptrs(__VA_ARGS__);                         \
        if (st_ != MOE_OK) return st_;                         \
    } while (0)

inline const bf16* cb(const void* p) { return static_cast<const bf16*>(p); }
inline bf16* mb(void* p) { return static_cast<bf16*>(p); }
inline cudaStream_t st(moe_stream_t s) { return static_cast<cudaStream_t>(s); }

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace
}  // namespace moe

using namespace moe;

extern "C" {

const char* moe_status_string(int status) {
    switch (status) {
        case MOE_OK: return "ok";
        case MOE_ERR_NULL: return "a required pointer is NULL";
        case MOE_ERR_DIMS: return "invalid dimensions";
        case MOE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (H, I must be multiples of 64; E <= 1024; K <= 32)";
        case MOE_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case MOE_ERR_WORKSPACE: return "workspace or arena too small";
        case MOE_ERR_CUDA: return "CUDA call failed";
        case MOE_ERR_BAD_INDEX: return "an expert id outside [0, E) was met (the pair was dropped)";
        case MOE_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        default: return "unknown status";
    }
}

size_t moe_permute_workspace_bytes(const moe_dims_t* dims) {
    if (check_dims(dims) != MOE_OK) return 0;
    return permute_workspace_bytes(*dims);
}

int moe_device_status(int* status_out) {
    if (status_out == nullptr) return MOE_ERR_NULL;
    return read_and_clear_device_status(status_out);
}

int moe_permute(const moe_dims_t* dims, const void* x, const int32_t* topk_idx, void* x_perm, int32_t* counts,
                int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row, void* workspace,
                size_t workspace_bytes, moe_stream_t stream) {
    {
        const void* const req[] = {topk_idx, counts, offsets, row_to_pair, pair_to_row, workspace};
        const void* const opt[] = {x, x_perm};
        MOE_VALIDATE(dims, req, opt);
    }
    if (x_perm != nullptr && x == nullptr) return MOE_ERR_NULL;
    if (workspace_bytes < permute_workspace_bytes(*dims)) return MOE_ERR_WORKSPACE;
    return launch_permute(*dims, cb(x), topk_idx, mb(x_perm), counts, offsets, row_to_pair, pair_to_row, workspace,
                          st(stream));
}

int moe_permute_static_scratch(const moe_dims_t* dims, const void* x, const int32_t* topk_idx, void* x_perm,
                               int32_t* counts, int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row,
                               moe_stream_t stream) {
    {
        const void* const req[] = {topk_idx, counts, offsets, row_to_pair, pair_to_row};
        const void* const opt[] = {x, x_perm};
        MOE_VALIDATE(dims, req, opt);
    }
    if (x_perm != nullptr && x == nullptr) return MOE_ERR_NULL;
    return launch_permute_static_scratch(*dims, cb(x), topk_idx, mb(x_perm), counts, offsets, row_to_pair,
                                         pair_to_row, st(stream));
}

int moe_permute_bwd(const moe_dims_t* dims, const void* dx_perm, const int32_t* pair_to_row, void* dx,
                    moe_stream_t stream) {
    const void* const req[] = {dx_perm, pair_to_row, dx};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_gather_sum(*dims, cb(dx_perm), nullptr, pair_to_row, mb(dx), st(stream));
}

int moe_grouped_gemm_gateup_swiglu(const moe_dims_t* dims, const void* x_perm, const void* w_gate, const void* w_up,
                                   const int32_t* offsets, void* h_act, void* gu_saved, moe_stream_t stream) {
    const void* const req[] = {x_perm, w_gate, w_up, offsets, h_act};
    const void* const opt[] = {gu_saved};
    MOE_VALIDATE(dims, req, opt);
    return launch_gateup_fwd(*dims, cb(x_perm), cb(w_gate), cb(w_up), offsets, mb(h_act), mb(gu_saved), st(stream));
}

int moe_grouped_gemm_down(const moe_dims_t* dims, const void* h_act, const void* w_down, const int32_t* offsets,
                          void* y_perm, moe_stream_t stream) {
    const void* const req[] = {h_act, w_down, offsets, y_perm};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_down_fwd(*dims, cb(h_act), cb(w_down), offsets, mb(y_perm), st(stream));
}

int moe_unpermute_combine(const moe_dims_t* dims, const void* y_perm, const float* topk_w, const int32_t* pair_to_row,
                          void* y, moe_stream_t stream) {
    const void* const req[] = {y_perm, topk_w, pair_to_row, y};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_gather_sum(*dims, cb(y_perm), topk_w, pair_to_row, mb(y), st(stream));
}

int moe_unpermute_combine_bwd(const moe_dims_t* dims, const void* dy, const void* y_perm, const float* topk_w,
                              const int32_t* pair_to_row, void* dy_perm, float* dtopk_w, moe_stream_t stream) {
    const void* const req[] = {dy, topk_w, pair_to_row, dy_perm};
    const void* const opt[] = {y_perm, dtopk_w};
    MOE_VALIDATE(dims, req, opt);
    if (dtopk_w != nullptr && y_perm == nullptr) return MOE_ERR_NULL;
    return launch_combine_bwd(*dims, cb(dy), cb(y_perm), topk_w, pair_to_row, mb(dy_perm), dtopk_w, st(stream));
}

int moe_grouped_gemm_down_dgrad(const moe_dims_t* dims, const void* dy_perm, const void* w_down,
                                const int32_t* offsets, void* dh_act, moe_stream_t stream) {
    const void* const req[] = {dy_perm, w_down, offsets, dh_act};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_down_dgrad(*dims, cb(dy_perm), cb(w_down), offsets, mb(dh_act), st(stream));
}

int moe_grouped_gemm_down_dgrad_swiglu_bwd(const moe_dims_t* dims, const void* dy_perm, const void* w_down,
                                           const void* gu_saved, const int32_t* offsets, void* dgu,
                                           moe_stream_t stream) {
    const void* const req[] = {dy_perm, w_down, gu_saved, offsets, dgu};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_down_dgrad_swiglu_bwd(*dims, cb(dy_perm), cb(w_down), cb(gu_saved), offsets, mb(dgu), st(stream));
}

int moe_grouped_gemm_down_wgrad(const moe_dims_t* dims, const void* h_act, const void* dy_perm,
                                const int32_t* offsets, void* dw_down, moe_stream_t stream) {
    const void* const req[] = {h_act, dy_perm, offsets, dw_down};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_down_wgrad(*dims, cb(h_act), cb(dy_perm), offsets, mb(dw_down), st(stream));
}

int moe_grouped_gemm_down_bwd(const moe_dims_t* dims, const void* dy_perm, const void* h_act, const void* w_down,
                              const int32_t* offsets, void* dh_act, void* dw_down, moe_stream_t stream) {
    int s = moe_grouped_gemm_down_dgrad(dims, dy_perm, w_down, offsets, dh_act, stream);
    if (s != MOE_OK) return s;
    return moe_grouped_gemm_down_wgrad(dims, h_act, dy_perm, offsets, dw_down, stream);
}

int moe_swiglu_bwd(const moe_dims_t* dims, const void* dh_act, const void* gu_saved, void* dgu,
                   moe_stream_t stream) {
    const void* const req[] = {dh_act, gu_saved, dgu};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_swiglu_bwd(*dims, cb(dh_act), cb(gu_saved), mb(dgu), st(stream));
}

int moe_grouped_gemm_gateup_dgrad(const moe_dims_t* dims, const void* dgu, const void* w_gate, const void* w_up,
                                  const int32_t* offsets, void* dx_perm, moe_stream_t stream) {
    const void* const req[] = {dgu, w_gate, w_up, offsets, dx_perm};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_gateup_dgrad(*dims, cb(dgu), cb(w_gate), cb(w_up), offsets, mb(dx_perm), st(stream));
}

int moe_grouped_gemm_gateup_wgrad(const moe_dims_t* dims, const void* x_perm, const void* dgu,
                                  const int32_t* offsets, void* dw_gate, void* dw_up, moe_stream_t stream) {
    const void* const req[] = {x_perm, dgu, offsets, dw_gate, dw_up};
    const void* const opt[] = {nullptr};
    MOE_VALIDATE(dims, req, opt);
    return launch_gateup_wgrad(*dims, cb(x_perm), cb(dgu), offsets, mb(dw_gate), mb(dw_up), st(stream));
}

int moe_grouped_gemm_gateup_swiglu_bwd(const moe_dims_t* dims, const void* dh_act, const void* gu_saved,
                                       const void* x_perm, const void* w_gate, const void* w_up,
                                       const int32_t* offsets, void* dgu, void* dx_perm, void* dw_gate,
                                       void* dw_up, moe_stream_t stream) {
    int s = moe_swiglu_bwd(dims, dh_act, gu_saved, dgu, stream);
    if (s != MOE_OK) return s;
    s = moe_grouped_gemm_gateup_dgrad(dims, dgu, w_gate, w_up, offsets, dx_perm, stream);
    if (s != MOE_OK) return s;
    return moe_grouped_gemm_gateup_wgrad(dims, x_perm, dgu, offsets, dw_gate, dw_up, stream);
}

// The router looks at T, E and K only.
static int check_router_dims(const moe_dims_t* d) {
    if (d == nullptr) return MOE_ERR_NULL;
    if (d->T <= 0 || d->E <= 0 || d->K <= 0 || d->K > d->E) return MOE_ERR_DIMS;
    if ((long long)d->T * d->K >= (1ll << 31)) return MOE_ERR_DIMS;
    if (d->E > 1024 || d->K > 32) return MOE_ERR_UNSUPPORTED_SHAPE;
    return MOE_OK;
}

int moe_router_topk(const moe_dims_t* dims, const float* logits, int32_t* topk_idx, float* topk_w,
                    moe_stream_t stream) {
    const void* const req[] = {logits, topk_idx, topk_w};
    const void* const opt[] = {nullptr};
    int st_ = check_router_dims(dims);
    if (st_ != MOE_OK) return st_;
    st_ = check_ptrs(req, opt);
    if (st_ != MOE_OK) return st_;
    return launch_router_topk(*dims, logits, topk_idx, topk_w, st(stream));
}

int moe_router_topk_bwd(const moe_dims_t* dims, const int32_t* topk_idx, const float* topk_w, const float* dtopk_w,
                        float* dlogits, moe_stream_t stream) {
    const void* const req[] = {topk_idx, topk_w, dtopk_w, dlogits};
    const void* const opt[] = {nullptr};
    int st_ = check_router_dims(dims);
    if (st_ != MOE_OK) return st_;
    st_ = check_ptrs(req, opt);
    if (st_ != MOE_OK) return st_;
    return launch_router_topk_bwd(*dims, topk_idx, topk_w, dtopk_w, dlogits, st(stream));
}

// ---- block-scaled FP8 down projection ----
static int check_mx_dims(const moe_dims_t* d) {
    const int st_ = check_dims(d);
    if (st_ != MOE_OK) return st_;
    return (d->H % 128 != 0 || d->I % 128 != 0) ? MOE_ERR_UNSUPPORTED_SHAPE : MOE_OK;
}

size_t moe_mxfp8_act_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return (size_t)(dims->I / 128) * (size_t)dims->T * dims->K * 4;
}

size_t moe_mxfp8_w_down_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return mx_w_scale_bytes(dims->E, dims->H, dims->I);
}

int moe_mxfp8_quantize_h_act(const moe_dims_t* dims, const void* h_act, void* codes, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {h_act, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_rows((long long)dims->T * dims->K, dims->I, cb(h_act), static_cast<uint8_t*>(codes),
                                   static_cast<uint8_t*>(scales), st(stream));
}

int moe_mxfp8_quantize_w_down(const moe_dims_t* dims, const void* w_down, void* codes_t, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {w_down, codes_t, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_w_transposed(dims->E, dims->I, dims->H, dims->H, 0, cb(w_down), static_cast<uint8_t*>(codes_t),
                                           static_cast<uint8_t*>(scales), st(stream));
}

int moe_grouped_gemm_down_mxfp8(const moe_dims_t* dims, const void* h_codes, const void* h_scales, const void* w_codes_t,
                                const void* w_scales, const int32_t* offsets, void* y_perm, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {h_codes, h_scales, w_codes_t, w_scales, offsets, y_perm};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_gemm((long long)dims->T * dims->K, dims->E, dims->H, dims->I, static_cast<const uint8_t*>(h_codes),
                          static_cast<const uint8_t*>(h_scales), static_cast<const uint8_t*>(w_codes_t),
                          static_cast<const uint8_t*>(w_scales), offsets, mb(y_perm), st(stream));
}

// ---- block-scaled FP8 data gradient of the down projection (contraction over H) ----
size_t moe_mxfp8_dy_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return (size_t)(dims->H / 128) * (size_t)dims->T * dims->K * 4;
}

size_t moe_mxfp8_w_down_dgrad_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return mx_w_scale_bytes(dims->E, dims->I, dims->H);
}

int moe_mxfp8_quantize_dy_perm(const moe_dims_t* dims, const void* dy_perm, void* codes, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {dy_perm, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_rows((long long)dims->T * dims->K, dims->H, cb(dy_perm), static_cast<uint8_t*>(codes),
                                   static_cast<uint8_t*>(scales), st(stream));
}

int moe_mxfp8_quantize_w_down_dgrad(const moe_dims_t* dims, const void* w_down, void* codes, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {w_down, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_w_rows(dims->E, dims->I, dims->H, dims->H, 0, cb(w_down), static_cast<uint8_t*>(codes),
                                     static_cast<uint8_t*>(scales), st(stream));
}

int moe_grouped_gemm_down_dgrad_mxfp8(const moe_dims_t* dims, const void* dy_codes, const void* dy_scales, const void* w_codes,
                                      const void* w_scales, const int32_t* offsets, void* dh_act, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {dy_codes, dy_scales, w_codes, w_scales, offsets, dh_act};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_gemm((long long)dims->T * dims->K, dims->E, dims->I, dims->H, static_cast<const uint8_t*>(dy_codes),
                          static_cast<const uint8_t*>(dy_scales), static_cast<const uint8_t*>(w_codes),
                          static_cast<const uint8_t*>(w_scales), offsets, mb(dh_act), st(stream));
}

// ---- block-scaled FP8 data gradient of the gate/up projection (contraction over the 2I gate and up features) ----
size_t moe_mxfp8_dgu_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return (size_t)(2 * dims->I / 128) * (size_t)dims->T * dims->K * 4;
}

size_t moe_mxfp8_w_gateup_dgrad_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return mx_w_scale_bytes(dims->E, dims->H, 2 * dims->I);
}

int moe_mxfp8_quantize_dgu(const moe_dims_t* dims, const void* dgu, void* codes, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {dgu, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_rows((long long)dims->T * dims->K, 2 * dims->I, cb(dgu), static_cast<uint8_t*>(codes),
                                   static_cast<uint8_t*>(scales), st(stream));
}

int moe_mxfp8_quantize_w_gateup_dgrad(const moe_dims_t* dims, const void* w_gate, const void* w_up, void* codes, void* scales,
                                      moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {w_gate, w_up, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    s = launch_mx_quantize_w_rows(dims->E, dims->H, dims->I, 2 * dims->I, 0, cb(w_gate), static_cast<uint8_t*>(codes),
                                  static_cast<uint8_t*>(scales), st(stream));
    if (s != MOE_OK) return s;
    return launch_mx_quantize_w_rows(dims->E, dims->H, dims->I, 2 * dims->I, dims->I, cb(w_up), static_cast<uint8_t*>(codes),
                                     static_cast<uint8_t*>(scales), st(stream));
}

int moe_grouped_gemm_gateup_dgrad_mxfp8(const moe_dims_t* dims, const void* dgu_codes, const void* dgu_scales, const void* w_codes,
                                        const void* w_scales, const int32_t* offsets, void* dx_perm, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {dgu_codes, dgu_scales, w_codes, w_scales, offsets, dx_perm};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_gemm((long long)dims->T * dims->K, dims->E, dims->H, 2 * dims->I, static_cast<const uint8_t*>(dgu_codes),
                          static_cast<const uint8_t*>(dgu_scales), static_cast<const uint8_t*>(w_codes),
                          static_cast<const uint8_t*>(w_scales), offsets, mb(dx_perm), st(stream));
}

// ---- block-scaled FP8 gate/up projection (contraction over H) and the SwiGLU activation with its quantiser ----
size_t moe_mxfp8_x_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return (size_t)(dims->H / 128) * (size_t)dims->T * dims->K * 4;
}

size_t moe_mxfp8_w_gateup_scale_bytes(const moe_dims_t* dims) {
    if (check_mx_dims(dims) != MOE_OK) return 0;
    return mx_w_scale_bytes(dims->E, 2 * dims->I, dims->H);
}

int moe_mxfp8_quantize_x_perm(const moe_dims_t* dims, const void* x_perm, void* codes, void* scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {x_perm, codes, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_rows((long long)dims->T * dims->K, dims->H, cb(x_perm), static_cast<uint8_t*>(codes),
                                   static_cast<uint8_t*>(scales), st(stream));
}

int moe_mxfp8_quantize_w_gateup(const moe_dims_t* dims, const void* w_gate, const void* w_up, void* codes_t, void* scales,
                                moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {w_gate, w_up, codes_t, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    s = launch_mx_quantize_w_transposed(dims->E, dims->H, dims->I, 2 * dims->I, 0, cb(w_gate), static_cast<uint8_t*>(codes_t),
                                        static_cast<uint8_t*>(scales), st(stream));
    if (s != MOE_OK) return s;
    return launch_mx_quantize_w_transposed(dims->E, dims->H, dims->I, 2 * dims->I, dims->I, cb(w_up), static_cast<uint8_t*>(codes_t),
                                           static_cast<uint8_t*>(scales), st(stream));
}

int moe_grouped_gemm_gateup_mxfp8(const moe_dims_t* dims, const void* x_codes, const void* x_scales, const void* w_codes_t,
                                  const void* w_scales, const int32_t* offsets, void* gu, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {x_codes, x_scales, w_codes_t, w_scales, offsets, gu};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_gemm((long long)dims->T * dims->K, dims->E, 2 * dims->I, dims->H, static_cast<const uint8_t*>(x_codes),
                          static_cast<const uint8_t*>(x_scales), static_cast<const uint8_t*>(w_codes_t),
                          static_cast<const uint8_t*>(w_scales), offsets, mb(gu), st(stream));
}

int moe_swiglu_mxfp8(const moe_dims_t* dims, const void* gu, void* h_act, void* h_codes, void* h_scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {gu, h_act, h_codes, h_scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_swiglu_quantize((long long)dims->T * dims->K, dims->I, cb(gu), mb(h_act), static_cast<uint8_t*>(h_codes),
                                     static_cast<uint8_t*>(h_scales), st(stream));
}

int moe_swiglu_bwd_mxfp8(const moe_dims_t* dims, const void* dh_act, const void* gu_saved, void* dgu, void* dgu_codes,
                         void* dgu_scales, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {dh_act, gu_saved, dgu, dgu_codes, dgu_scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_swiglu_bwd_quantize((long long)dims->T * dims->K, dims->I, cb(dh_act), cb(gu_saved), mb(dgu),
                                         static_cast<uint8_t*>(dgu_codes), static_cast<uint8_t*>(dgu_scales), st(stream));
}

// ---- block-scaled FP8 weight gradients (contraction over the packed rows of each expert) ----
static int check_tokens_args(const moe_dims_t* d, int n_features) {
    const int s = check_mx_dims(d);
    if (s != MOE_OK) return s;
    return (n_features <= 0 || n_features % 128 != 0) ? MOE_ERR_UNSUPPORTED_SHAPE : MOE_OK;
}

size_t moe_mxfp8_tokens_codes_bytes(const moe_dims_t* dims, int n_features) {
    if (check_tokens_args(dims, n_features) != MOE_OK) return 0;
    return (size_t)n_features * (size_t)mx_tokens_pitch((long long)dims->T * dims->K, dims->E);
}

size_t moe_mxfp8_tokens_scale_bytes(const moe_dims_t* dims, int n_features) {
    if (check_tokens_args(dims, n_features) != MOE_OK) return 0;
    return mx_tokens_scale_bytes((long long)dims->T * dims->K, dims->E, n_features);
}

int moe_mxfp8_quantize_tokens(const moe_dims_t* dims, const void* x, int ld, int col0, int n_features, const int32_t* offsets,
                              void* codes_t, void* scales, moe_stream_t stream) {
    int s = check_tokens_args(dims, n_features);
    if (s != MOE_OK) return s;
    if (ld <= 0 || col0 < 0 || col0 % 8 != 0 || ld % 8 != 0 || col0 + n_features > ld) return MOE_ERR_DIMS;
    const void* const req[] = {x, offsets, codes_t, scales};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_quantize_tokens((long long)dims->T * dims->K, dims->E, cb(x), ld, col0, n_features, offsets,
                                     static_cast<uint8_t*>(codes_t), static_cast<uint8_t*>(scales), st(stream));
}

int moe_grouped_gemm_down_wgrad_mxfp8(const moe_dims_t* dims, const void* h_codes_t, const void* h_scales, const void* dy_codes_t,
                                      const void* dy_scales, void* dw_down, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {h_codes_t, h_scales, dy_codes_t, dy_scales, dw_down};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    return launch_mx_wgrad((long long)dims->T * dims->K, dims->E, dims->I, dims->H, static_cast<const uint8_t*>(h_codes_t),
                           static_cast<const uint8_t*>(h_scales), static_cast<const uint8_t*>(dy_codes_t),
                           static_cast<const uint8_t*>(dy_scales), mb(dw_down), st(stream));
}

int moe_grouped_gemm_gateup_wgrad_mxfp8(const moe_dims_t* dims, const void* x_codes_t, const void* x_scales,
                                        const void* dg_codes_t, const void* dg_scales, const void* du_codes_t,
                                        const void* du_scales, void* dw_gate, void* dw_up, moe_stream_t stream) {
    int s = check_mx_dims(dims);
    if (s != MOE_OK) return s;
    const void* const req[] = {x_codes_t, x_scales, dg_codes_t, dg_scales, du_codes_t, du_scales, dw_gate, dw_up};
    const void* const opt[] = {nullptr};
    s = check_ptrs(req, opt);
    if (s != MOE_OK) return s;
    const long long R = (long long)dims->T * dims->K;
    s = launch_mx_wgrad(R, dims->E, dims->H, dims->I, static_cast<const uint8_t*>(x_codes_t), static_cast<const uint8_t*>(x_scales),
                        static_cast<const uint8_t*>(dg_codes_t), static_cast<const uint8_t*>(dg_scales), mb(dw_gate), st(stream));
    if (s != MOE_OK) return s;
    return launch_mx_wgrad(R, dims->E, dims->H, dims->I, static_cast<const uint8_t*>(x_codes_t), static_cast<const uint8_t*>(x_scales),
                           static_cast<const uint8_t*>(du_codes_t), static_cast<const uint8_t*>(du_scales), mb(dw_up), st(stream));
}

// Arena layout of moe_layer_fwd_bwd_host (every block 256-byte aligned).
namespace {
// Two side streams (uploads, downloads) and a few events per device for moe_layer_fwd_bwd_host, created on first
// use and kept for the life of the process (the one place where the library creates CUDA objects of its own).
struct HostCopyLane {
    cudaStream_t stream;      // downloads
    cudaStream_t up_stream;   // uploads
    cudaEvent_t begin, x_up, dy_up, y_ready, dx_ready, down_done, inputs_free;
    bool ready;
    bool primed;              // inputs_free has been recorded by an earlier call
};
HostCopyLane* host_copy_lane() {
    static HostCopyLane lanes[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostCopyLane& l = lanes[dev];
    if (!l.ready) {
        if (cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&l.up_stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        cudaEvent_t* evs[7] = {&l.begin, &l.x_up, &l.dy_up, &l.y_ready, &l.dx_ready, &l.down_done, &l.inputs_free};
        for (cudaEvent_t* e : evs)
            if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        l.ready = true;
    }
    return &l;
}
struct Arena {
    size_t x, idx, w, dy, y, dx, dw, counts, offsets, r2p, p2r, ws, xp, hact, gu, yp, dyp, dhact, dgu, dxp, total;
};
Arena arena_layout(const moe_dims_t& d) {
    const size_t T = d.T, H = d.H, I = d.I, E = d.E, K = d.K, R = T * K;
    Arena a;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    a.x = take(T * H * 2); a.idx = take(R * 4); a.w = take(R * 4); a.dy = take(T * H * 2);
    a.y = take(T * H * 2); a.dx = take(T * H * 2); a.dw = take(R * 4);
    a.counts = take(E * 4); a.offsets = take((E + 1) * 4); a.r2p = take(R * 4); a.p2r = take(R * 4);
    a.ws = take(permute_workspace_bytes(d));
    a.xp = take(R * H * 2); a.hact = take(R * I * 2); a.gu = take(R * 2 * I * 2); a.yp = take(R * H * 2);
    a.dyp = take(R * H * 2); a.dhact = take(R * I * 2); a.dgu = take(R * 2 * I * 2); a.dxp = take(R * H * 2);
    a.total = o;
    return a;
}
}  // namespace

size_t moe_layer_arena_bytes(const moe_dims_t* dims) {
    if (check_dims(dims) != MOE_OK) return 0;
    return arena_layout(*dims).total;
}

int moe_layer_fwd_bwd_host(const moe_dims_t* dims, const void* x_host, const int32_t* topk_idx_host,
                           const float* topk_w_host, const void* dy_host, const void* w_gate, const void* w_up,
                           const void* w_down, void* y_host, void* dx_host, float* dtopk_w_host, void* dw_gate,
                           void* dw_up, void* dw_down, void* arena, size_t arena_bytes, moe_stream_t stream) {
    {
        const void* const req[] = {w_gate, w_up, w_down, dw_gate, dw_up, dw_down, arena};
        const void* const opt[] = {nullptr};
        MOE_VALIDATE(dims, req, opt);
    }
    if (!x_host || !topk_idx_host || !topk_w_host || !dy_host || !y_host || !dx_host || !dtopk_w_host)
        return MOE_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return MOE_ERR_ALIGNMENT;
    const moe_dims_t& d = *dims;
    const Arena a = arena_layout(d);
    if (arena_bytes < a.total) return MOE_ERR_WORKSPACE;
    uint8_t* base = static_cast<uint8_t*>(arena);
    cudaStream_t s = st(stream);
    const size_t T = d.T, H = d.H, R = T * d.K;
    auto P = [&](size_t off) { return static_cast<void*>(base + off); };
    auto Pi = [&](size_t off) { return reinterpret_cast<int32_t*>(base + off); };

    // Side streams for the copies, so that they overlap compute: y comes down while the backward pass runs, dx and
    // dtopk_w come down under the two weight-gradient GEMMs, and the uploads of a call wait only until the PREVIOUS
    // call's last reader of the input blocks of the arena (its combine-backward) is done -- when calls follow one
    // another, the next call's x, routing and dy travel to the device under this call's backward GEMMs.  The first
    // call on a device orders its uploads after everything already on the caller's stream.  Everything else is
    // ordered against the caller's stream with events.
    HostCopyLane* lane = host_copy_lane();
    if (lane == nullptr) return MOE_ERR_CUDA;
    cudaStream_t c = lane->stream, u = lane->up_stream;
    if (lane->primed) {
        if (cudaStreamWaitEvent(u, lane->inputs_free, 0) != cudaSuccess) return MOE_ERR_CUDA;
    } else {
        if (cudaEventRecord(lane->begin, s) != cudaSuccess || cudaStreamWaitEvent(u, lane->begin, 0) != cudaSuccess)
            return MOE_ERR_CUDA;
    }
    if (cudaMemcpyAsync(P(a.x), x_host, T * H * 2, cudaMemcpyHostToDevice, u) != cudaSuccess ||
        cudaMemcpyAsync(P(a.idx), topk_idx_host, R * 4, cudaMemcpyHostToDevice, u) != cudaSuccess ||
        cudaMemcpyAsync(P(a.w), topk_w_host, R * 4, cudaMemcpyHostToDevice, u) != cudaSuccess ||
        cudaEventRecord(lane->x_up, u) != cudaSuccess ||
        cudaMemcpyAsync(P(a.dy), dy_host, T * H * 2, cudaMemcpyHostToDevice, u) != cudaSuccess ||
        cudaEventRecord(lane->dy_up, u) != cudaSuccess || cudaStreamWaitEvent(s, lane->x_up, 0) != cudaSuccess)
        return MOE_ERR_CUDA;

    int rc;
#define MOE_STEP(call) do { rc = (call); if (rc != MOE_OK) return rc; } while (0)
    MOE_STEP(moe_permute(dims, P(a.x), Pi(a.idx), P(a.xp), Pi(a.counts), Pi(a.offsets), Pi(a.r2p), Pi(a.p2r), P(a.ws),
                         a.xp - a.ws, stream));
    MOE_STEP(moe_grouped_gemm_gateup_swiglu(dims, P(a.xp), w_gate, w_up, Pi(a.offsets), P(a.hact), P(a.gu), stream));
    MOE_STEP(moe_grouped_gemm_down(dims, P(a.hact), w_down, Pi(a.offsets), P(a.yp), stream));
    MOE_STEP(moe_unpermute_combine(dims, P(a.yp), reinterpret_cast<float*>(base + a.w), Pi(a.p2r), P(a.y), stream));
    if (cudaEventRecord(lane->y_ready, s) != cudaSuccess || cudaStreamWaitEvent(c, lane->y_ready, 0) != cudaSuccess ||
        cudaMemcpyAsync(y_host, P(a.y), T * H * 2, cudaMemcpyDeviceToHost, c) != cudaSuccess ||
        cudaStreamWaitEvent(s, lane->dy_up, 0) != cudaSuccess)
        return MOE_ERR_CUDA;
    MOE_STEP(moe_unpermute_combine_bwd(dims, P(a.dy), P(a.yp), reinterpret_cast<float*>(base + a.w), Pi(a.p2r),
                                       P(a.dyp), reinterpret_cast<float*>(base + a.dw), stream));
    // x, routing and dy have been read for the last time: a following call may overwrite them from here on
    if (cudaEventRecord(lane->inputs_free, s) != cudaSuccess) return MOE_ERR_CUDA;
    lane->primed = true;
    // backward in pieces: the whole data-gradient chain first, so that dx can travel to the host while the two
    // weight-gradient GEMMs (which nothing downstream waits for) are still running
    MOE_STEP(moe_grouped_gemm_down_dgrad(dims, P(a.dyp), w_down, Pi(a.offsets), P(a.dhact), stream));
    MOE_STEP(moe_swiglu_bwd(dims, P(a.dhact), P(a.gu), P(a.dgu), stream));
    MOE_STEP(moe_grouped_gemm_gateup_dgrad(dims, P(a.dgu), w_gate, w_up, Pi(a.offsets), P(a.dxp), stream));
    MOE_STEP(moe_permute_bwd(dims, P(a.dxp), Pi(a.p2r), P(a.dx), stream));
    if (cudaEventRecord(lane->dx_ready, s) != cudaSuccess || cudaStreamWaitEvent(c, lane->dx_ready, 0) != cudaSuccess ||
        cudaMemcpyAsync(dx_host, P(a.dx), T * H * 2, cudaMemcpyDeviceToHost, c) != cudaSuccess ||
        cudaMemcpyAsync(dtopk_w_host, P(a.dw), R * 4, cudaMemcpyDeviceToHost, c) != cudaSuccess ||
        cudaEventRecord(lane->down_done, c) != cudaSuccess)
        return MOE_ERR_CUDA;
    MOE_STEP(moe_grouped_gemm_down_wgrad(dims, P(a.hact), P(a.dyp), Pi(a.offsets), dw_down, stream));
    MOE_STEP(moe_grouped_gemm_gateup_wgrad(dims, P(a.xp), P(a.dgu), Pi(a.offsets), dw_gate, dw_up, stream));
#undef MOE_STEP

    // the caller's stream also covers the side copies (y, then dx and dtopk_w, in stream order on the side stream)
    if (cudaStreamWaitEvent(s, lane->down_done, 0) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
}

}  // extern "C"
