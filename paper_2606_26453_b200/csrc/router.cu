// Router in front of the layer: per token, the K largest of E logits (descending, equal values to the lower
// expert id) and the softmax over the kept logits (= the full softmax renormalised over the kept experts),
// plus the backward from the weight gradients to the logits.  The benchmark workloads describe this step as
// how their routing inputs are made; the paper has no counterpart.
//
// One warp per token.  The E <= 1024 logits of a row sit in registers, element e = j*32 + lane (coalesced
// loads).  Selection is K rounds of: per-lane best among the not-yet-taken elements, then a warp arg-max with
// two integer redux instructions (maximum of an order-preserving key, then the lowest id among its holders).
// All comparisons are on the float32 values as given, so the indices are exact.
// HBM-bound in principle (T*E*4 bytes in, 8*T*K out), in practice a few microseconds.
#include <limits.h>
#include <math.h>

#include "common.cuh"

namespace moe {
namespace {

constexpr int kWarpsPerBlock = 8;

// Order-preserving map of a float onto unsigned integers (larger float <=> larger key; -inf maps above 0, which
// stands for "no candidate"), and its inverse.  Lets the warp arg-max run on the integer redux instructions.
__device__ __forceinline__ uint32_t key_of(float v) {
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float value_of(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

template <int VPL>   // logits per lane, E <= 32 * VPL
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
router_topk_kernel(const float* __restrict__ logits, int T, int E, int K, int32_t* __restrict__ topk_idx,
                   float* __restrict__ topk_w) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (t >= T) return;
    const float* row = logits + (size_t)t * E;
    uint32_t key[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int e = j * 32 + lane;
        key[j] = e < E ? key_of(row[e] + 0.0f) : 0u;   // + 0.0f: -0.0 and +0.0 compare equal, so they share a key
    }
    float my_val = 0.f;                 // lane k keeps the k-th selection
    int my_idx = 0;
    for (int k = 0; k < K; ++k) {
        // this lane's best remaining element (ascending j = ascending id, strict > keeps the lower id on ties)
        uint32_t bk = 0u;
        int bj = 0;
#pragma unroll
        for (int j = 0; j < VPL; ++j)
            if (key[j] > bk) { bk = key[j]; bj = j; }
        const uint32_t kmax = __reduce_max_sync(0xffffffffu, bk);
        // among the lanes that hold the maximum: the lowest expert id
        const uint32_t cand = (bk == kmax && bk != 0u) ? (uint32_t)(bj * 32 + lane) : 0xffffffffu;
        const uint32_t imin = __reduce_min_sync(0xffffffffu, cand);
        if ((int)(imin & 31u) == lane && imin != 0xffffffffu) {
#pragma unroll
            for (int j = 0; j < VPL; ++j)
                if (j == (int)(imin >> 5)) key[j] = 0u;   // taken
        }
        if (k == lane) { my_val = value_of(kmax); my_idx = (int)imin; }
    }
    // softmax over the kept logits; the first selection is the row maximum
    const float m = __shfl_sync(0xffffffffu, my_val, 0);
    float ex = lane < K ? expf(my_val - m) : 0.f;
    float sum = ex;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane < K) {
        topk_idx[(size_t)t * K + lane] = my_idx;
        topk_w[(size_t)t * K + lane] = ex / sum;
    }
}

// dz[t, idx_k] = w_k (dw_k - sum_j w_j dw_j); zero elsewhere.  One warp per token.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
router_topk_bwd_kernel(const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_w,
                       const float* __restrict__ dtopk_w, int T, int E, int K, float* __restrict__ dlogits) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (t >= T) return;
    float w = 0.f, dw = 0.f;
    int idx = -1;
    if (lane < K) {
        idx = topk_idx[(size_t)t * K + lane];
        w = topk_w[(size_t)t * K + lane];
        dw = dtopk_w[(size_t)t * K + lane];
    }
    float inner = w * dw;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) inner += __shfl_xor_sync(0xffffffffu, inner, off);
    float* row = dlogits + (size_t)t * E;
    for (int e = lane; e < E; e += 32) row[e] = 0.f;
    __syncwarp();   // orders the zero fill before the K scattered values of the same warp
    if (lane < K && idx >= 0 && idx < E) row[idx] = w * (dw - inner);
}

}  // namespace

int launch_router_topk(const moe_dims_t& d, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t s) {
    const int blocks = (d.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int vpl = (d.E + 31) / 32;
#define MOE_ROUTER_CASE(V)                                                                                     \
    if (vpl <= V) {                                                                                            \
        router_topk_kernel<V><<<blocks, kWarpsPerBlock * 32, 0, s>>>(logits, d.T, d.E, d.K, topk_idx, topk_w); \
        return check_launch();                                                                                 \
    }
    MOE_ROUTER_CASE(1)
    MOE_ROUTER_CASE(2)
    MOE_ROUTER_CASE(4)
    MOE_ROUTER_CASE(8)
    MOE_ROUTER_CASE(16)
    MOE_ROUTER_CASE(32)
#undef MOE_ROUTER_CASE
    return MOE_ERR_UNSUPPORTED_SHAPE;
}

int launch_router_topk_bwd(const moe_dims_t& d, const int32_t* topk_idx, const float* topk_w, const float* dtopk_w,
                           float* dlogits, cudaStream_t s) {
    const int blocks = (d.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    router_topk_bwd_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(topk_idx, topk_w, dtopk_w, d.T, d.E, d.K, dlogits);
    return check_launch();
}

}  // namespace moe
