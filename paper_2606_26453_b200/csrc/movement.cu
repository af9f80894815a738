// HBM-bound kernels of the MoE layer: route-permute (stable counting sort by expert + row
// gather), unpermute-combine and its backward, permute backward, SwiGLU backward.
//
// Row movement is token-major: every source row is read once and written (bulk copies) or gathered
// (16-byte loads) K times, so the bytes moved are the algorithmic minimum.  The permutation indices
// never depend on the order in which atomics land: ranks come from warp-level match/ballot
// scans over pairs taken in ascending pair id, which makes the result the unique stable sort.
#include "common.cuh"

namespace moe {

namespace {

constexpr int kWorkspacePairsPerRow = 256;   // the workspace holds one histogram row per 256 pairs (an upper bound on what is used)
constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;

__device__ __forceinline__ uint4 ldg16(const uint4* p) { return __ldg(p); }

__device__ __forceinline__ void unpack8(const uint4& v, float f[8]) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 t = __bfloat1622float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

__device__ __forceinline__ uint4 pack8(const float f[8]) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
}

// ------------------------------------------------------------------------------------------------
// a1, index part.  Two small kernels over the R = T*K pairs, split into block-chunks of `chunk`
// consecutive pairs (a multiple of 256; one block per chunk, one eighth of it per warp):
//   hist : per block-chunk, the number of pairs of each expert (shared-memory atomics: counts are
//          order-free)                                                          -> ws[block][e]
//   rank : every block sums the histogram rows before it (its base) and all rows (the counts),
//          turns the counts into offsets, ranks its warps' pairs (per-warp counts by atomics, then the
//          same-expert lane mask of each 32 pairs from 32 broadcasts, and popc):
//          row(p) = offsets[e] + base[e] + pairs of e in earlier warps of the block + earlier
//          pairs of e in the same warp.
// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch: the three permute kernels are launched so that a later one may start (and run its
// set-up) while the earlier one is still finishing; grid_dependency_wait() then blocks until everything the earlier
// kernel wrote is visible.  Saves the launch gaps of the two small index kernels.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr int kIdxGroup = 8;   // index loads in flight per thread in the permute index kernels

__global__ void __launch_bounds__(kThreads) permute_hist_kernel(const int32_t* __restrict__ topk_idx, int R, int E,
                                                                int chunk, int32_t* __restrict__ ws) {
    extern __shared__ int32_t smem_i[];
    int32_t* hist = smem_i;   // [E]
    grid_launch_dependents();
    for (int e = threadIdx.x; e < E; e += kThreads) hist[e] = 0;
    __syncthreads();
    const long long p0 = (long long)blockIdx.x * chunk;
    // chunk is a multiple of kThreads: whole warps stay together.  The indices of kIdxGroup iterations are loaded
    // first, so that their global-memory latencies overlap instead of adding up one after the other.
    for (int i0 = threadIdx.x; i0 < chunk; i0 += kThreads * kIdxGroup) {
        int ev[kIdxGroup];
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            const int i = i0 + g * kThreads;
            const long long p = p0 + i;
            int e = (i < chunk && p < R) ? topk_idx[p] : -1;
            ev[g] = e >= E ? -1 : e;
        }
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            if (i0 - (int)threadIdx.x + g * kThreads >= chunk) break;   // block-uniform
            if (ev[g] >= 0) atomicAdd(&hist[ev[g]], 1);   // counts only: order-free
        }
    }
    __syncthreads();
    int32_t* out = ws + (size_t)blockIdx.x * E;
    for (int e = threadIdx.x; e < E; e += kThreads) out[e] = hist[e];
}

__global__ void __launch_bounds__(kThreads) permute_rank_kernel(const int32_t* __restrict__ topk_idx, int R, int E,
                                                                int chunk, int n_blocks,
                                                                const int32_t* __restrict__ ws,
                                                                int32_t* __restrict__ counts,
                                                                int32_t* __restrict__ offsets,
                                                                int32_t* __restrict__ row_to_pair,
                                                                int32_t* __restrict__ pair_to_row) {
    extern __shared__ int32_t smem_i[];
    int32_t* offs = smem_i;                       // [E+1] exclusive prefix of the counts
    int32_t* total = smem_i + (E + 1);            // [E]   counts
    int32_t* base = total + E;                    // [E]   pairs of e in earlier blocks
    int32_t* whist = base + E;                    // [warps][E] per-warp counts, then running row cursors
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Before the histogram kernel's output is needed: this warp's own counts over its eighth of the chunk (pass 1,
    // from the routing indices alone).
    grid_launch_dependents();
    for (int i = threadIdx.x; i < kWarpsPerBlock * E; i += kThreads) whist[i] = 0;
    __syncthreads();
    // pass 1: this warp's histogram over its eighth of the chunk
    const int per_warp = chunk / kWarpsPerBlock;
    const long long p0 = (long long)blockIdx.x * chunk + (long long)warp * per_warp;
    int32_t* mine = whist + warp * E;
#pragma unroll 1
    for (int i0 = 0; i0 < per_warp; i0 += 32 * kIdxGroup) {   // indices of kIdxGroup iterations loaded up front
        int ev[kIdxGroup];
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            const int i = i0 + g * 32 + lane;
            const long long p = p0 + i;
            int e = (i < per_warp && p < R) ? topk_idx[p] : -1;
            ev[g] = e >= E ? -1 : e;
        }
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            if (i0 + g * 32 >= per_warp) break;   // warp-uniform
            if (ev[g] >= 0) atomicAdd(&mine[ev[g]], 1);   // counts only: order-free
        }
    }
    grid_dependency_wait();   // the per-block histograms of the first kernel are complete and visible from here on
    for (int e = threadIdx.x; e < E; e += kThreads) {
        int before = 0, all = 0;
        for (int b = 0; b < n_blocks; ++b) {
            const int v = ws[(size_t)b * E + e];
            all += v;
            if (b < (int)blockIdx.x) before += v;
        }
        total[e] = all;
        base[e] = before;
    }
    __syncthreads();
    // offsets = exclusive prefix of counts, by warp 0 (each lane owns a contiguous run of experts)
    if (warp == 0) {
        const int per = (E + 31) / 32;
        const int e0 = min(lane * per, E), e1 = min(e0 + per, E);
        int sum = 0;
        for (int e = e0; e < e1; ++e) sum += total[e];
        int incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        int run = incl - sum;
        for (int e = e0; e < e1; ++e) {
            offs[e] = run;
            run += total[e];
        }
        if (lane == 31) offs[E] = incl;
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        for (int e = threadIdx.x; e <= E; e += kThreads) offsets[e] = offs[e];
        for (int e = threadIdx.x; e < E; e += kThreads) counts[e] = total[e];
    }
    // per-warp counts -> first row of each (warp, expert)
    for (int e = threadIdx.x; e < E; e += kThreads) {
        int run = offs[e] + base[e];
#pragma unroll
        for (int w = 0; w < kWarpsPerBlock; ++w) {
            const int v = whist[w * E + e];
            whist[w * E + e] = run;
            run += v;
        }
    }
    __syncthreads();
    // pass 2: stable ranks
    const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll 1
    for (int i0 = 0; i0 < per_warp; i0 += 32 * kIdxGroup) {
        int ev[kIdxGroup];
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            const int i = i0 + g * 32 + lane;
            const long long p = p0 + i;
            int e = (i < per_warp && p < R) ? topk_idx[p] : -1;
            ev[g] = e >= E ? -1 : e;
        }
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            if (i0 + g * 32 >= per_warp) break;   // warp-uniform
            const int e = ev[g];
            const long long p = p0 + i0 + g * 32 + lane;
            // lanes of the warp with the same expert: 32 broadcasts are several times faster than match.any here
            // (whose time grows with the number of distinct values, and routing makes most of them distinct)
            unsigned mask = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) mask |= (__shfl_sync(0xffffffffu, e, j) == e ? 1u : 0u) << j;
            if (e >= 0) {
                const int row = mine[e] + __popc(mask & lt_mask);
                row_to_pair[row] = (int32_t)p;
                pair_to_row[p] = row;
            }
            __syncwarp();
            if (e >= 0 && lane == __ffs(mask) - 1) mine[e] += __popc(mask);
            __syncwarp();
        }
    }
}

// ------------------------------------------------------------------------------------------------
// a1, row part: x_perm[pair_to_row[t*K+k], :] = x[t, :] with the bulk-copy engine.  One warp per CTA
// runs a ring of NBUF shared-memory buffers: a token row (or a <= 16 KB segment of it) is pulled in
// with one cp.async.bulk load and pushed to its K destination rows with K cp.async.bulk stores
// (lane k issues store k), so the row is read from HBM once and no data passes through registers.
// Loads run kRowLookahead units ahead of the stores.
// ------------------------------------------------------------------------------------------------
constexpr int kRowBufs = 4, kRowLookahead = 2, kRowMaxSeg = 16384;
__device__ int g_movement_status = 0;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(32) permute_rows_bulk_kernel(const uint8_t* __restrict__ x,
                                                               const int32_t* __restrict__ pair_to_row,
                                                               uint8_t* __restrict__ x_perm, int T, int K,
                                                               int row_bytes, int seg_bytes, int n_seg) {
    extern __shared__ __align__(128) uint8_t bufs[];   // [kRowBufs][seg_bytes]
    __shared__ unsigned long long bars[kRowBufs];
    __shared__ int32_t dest[kRowBufs][32];
    const int lane = threadIdx.x;
    if (lane == 0) {
        for (int s = 0; s < kRowBufs; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[s])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    grid_dependency_wait();   // pair_to_row comes from the rank kernel, which may still be finishing
    const long long n_units_all = (long long)T * n_seg;
    const long long first = blockIdx.x, stride = gridDim.x;
    const long long n_mine = first < n_units_all ? (n_units_all - first + stride - 1) / stride : 0;
    bool ok = true;
    for (long long it = 0; ok && it < n_mine + kRowLookahead; ++it) {
        if (it < n_mine) {
            const int s = (int)(it % kRowBufs);
            const long long u = first + it * stride;
            const int t = (int)(u / n_seg), seg = (int)(u - (long long)t * n_seg);
            const int bytes = min(seg_bytes, row_bytes - seg * seg_bytes);
            // the stores that last read this buffer were committed kRowLookahead iterations ago
            if (it >= kRowBufs) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kRowLookahead - 1) : "memory");
            if (lane < K) dest[s][lane] = __ldg(pair_to_row + (long long)t * K + lane);
            __syncwarp();
            if (lane == 0) {
                const uint32_t bar = smem_addr(&bars[s]);
                asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes)
                             : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                                 smem_addr(bufs + (size_t)s * seg_bytes)),
                             "l"(x + (long long)t * row_bytes + (long long)seg * seg_bytes), "r"(bytes), "r"(bar)
                             : "memory");
            }
        }
        const long long j = it - kRowLookahead;
        if (j >= 0) {
            const int s = (int)(j % kRowBufs);
            const uint32_t parity = (uint32_t)((j / kRowBufs) & 1);
            const long long u = first + j * stride;
            const int t = (int)(u / n_seg), seg = (int)(u - (long long)t * n_seg);
            const int bytes = min(seg_bytes, row_bytes - seg * seg_bytes);
            const uint32_t bar = smem_addr(&bars[s]);
            uint32_t done = 0;
            for (uint32_t spin = 0; !done; ++spin) {
                asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                             : "=r"(done)
                             : "r"(bar), "r"(parity)
                             : "memory");
                if (!done && spin > (1u << 24)) {   // bounded: give up, report, leave
                    atomicExch(&g_movement_status, (int)MOE_ERR_TIMEOUT);
                    ok = false;
                    break;
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane < K) {
                uint8_t* dst = x_perm + (long long)dest[s][lane] * row_bytes + (long long)seg * seg_bytes;
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
                             "r"(smem_addr(bufs + (size_t)s * seg_bytes)), "r"(bytes)
                             : "memory");
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
}

// ------------------------------------------------------------------------------------------------
// a4 / a8: dst[t,:] = sum_k w[t,k] * src[pair_to_row[t*K+k], :]  (w == NULL: unit weights).
// fp32 accumulation in slot order, one rounding to bf16.
// ------------------------------------------------------------------------------------------------
template <int KT, bool WEIGHTED>
__global__ void __launch_bounds__(kThreads) gather_sum_kernel(const uint4* __restrict__ src,
                                                              const float* __restrict__ topk_w,
                                                              const int32_t* __restrict__ pair_to_row,
                                                              uint4* __restrict__ dst, long long total, int hv,
                                                              int K) {
    const long long i = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (i >= total) return;
    const int t = (int)(i / hv);
    const int c = (int)(i - (long long)t * hv);
    const int32_t* rows = pair_to_row + (long long)t * K;
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
    if (KT > 0) {
        uint4 v[KT > 0 ? KT : 1];
        float w[KT > 0 ? KT : 1];
#pragma unroll
        for (int k = 0; k < KT; ++k) {
            v[k] = ldg16(src + (long long)__ldg(rows + k) * hv + c);
            w[k] = WEIGHTED ? __ldg(topk_w + (long long)t * K + k) : 1.f;
        }
#pragma unroll
        for (int k = 0; k < KT; ++k) {
            float f[8];
            unpack8(v[k], f);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = WEIGHTED ? fmaf(w[k], f[j], acc[j]) : acc[j] + f[j];
        }
    } else {
        for (int k = 0; k < K; ++k) {
            const uint4 v = ldg16(src + (long long)__ldg(rows + k) * hv + c);
            const float w = WEIGHTED ? __ldg(topk_w + (long long)t * K + k) : 1.f;
            float f[8];
            unpack8(v, f);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = WEIGHTED ? fmaf(w, f[j], acc[j]) : acc[j] + f[j];
        }
    }
    dst[i] = pack8(acc);
}

// ------------------------------------------------------------------------------------------------
// a5: one block per token, one thread per 16-byte piece of the row.
// dy_perm[row_k, :] = w_k * dy[t, :]; dtopk_w[t,k] = <dy[t,:], y_perm[row_k,:]> (warp shuffles, then a
// fixed-order sum over the block's warps: deterministic).  y_perm pieces are fetched four slots at a time
// to keep the register count low enough for five blocks per SM.
// ------------------------------------------------------------------------------------------------
template <int KT, bool WITH_DW>
__global__ void __launch_bounds__(kThreads, 5) combine_bwd_kernel(const uint4* __restrict__ dy,
                                                                  const uint4* __restrict__ y_perm,
                                                                  const float* __restrict__ topk_w,
                                                                  const int32_t* __restrict__ pair_to_row,
                                                                  uint4* __restrict__ dy_perm,
                                                                  float* __restrict__ dtopk_w, int T, int hv, int K) {
    constexpr int KA = KT > 0 ? KT : 32;
    __shared__ float partial[kWarpsPerBlock][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x;
    const int kk = KT > 0 ? KT : K;
    const int32_t* rows = pair_to_row + (long long)t * K;
    const float* wt = topk_w + (long long)t * K;
    float dot[KA];
#pragma unroll
    for (int k = 0; k < KA; ++k) dot[k] = 0.f;
    for (int c = threadIdx.x; c < hv; c += kThreads) {
        const uint4 dv = ldg16(dy + (long long)t * hv + c);
        float d[8];
        unpack8(dv, d);
#pragma unroll
        for (int k0 = 0; k0 < KA; k0 += 4) {
            uint4 yv[4];
            long long row[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (k0 + q < kk) {
                    row[q] = __ldg(rows + k0 + q);
                    if (WITH_DW) yv[q] = ldg16(y_perm + row[q] * hv + c);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (k0 + q < kk) {
                    const float w = __ldg(wt + k0 + q);
                    float o[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) o[j] = w * d[j];
                    dy_perm[row[q] * hv + c] = pack8(o);
                    if (WITH_DW) {
                        float y[8];
                        unpack8(yv[q], y);
#pragma unroll
                        for (int j = 0; j < 8; ++j) dot[k0 + q] = fmaf(d[j], y[j], dot[k0 + q]);
                    }
                }
            }
        }
    }
    if (WITH_DW) {
#pragma unroll
        for (int k = 0; k < KA; ++k) {
            if (k < kk) {
                float v = dot[k];
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
                if (lane == 0) partial[warp][k] = v;
            }
        }
        __syncthreads();
        if (threadIdx.x < kk) {
            float v = 0.f;
#pragma unroll
            for (int wq = 0; wq < kWarpsPerBlock; ++wq) v += partial[wq][threadIdx.x];
            dtopk_w[(long long)t * K + threadIdx.x] = v;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// a7, elementwise part: dGU = [dg | du] from dHact and the saved pre-activations [g | u].
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) swiglu_bwd_kernel(const uint4* __restrict__ dh_act,
                                                              const uint4* __restrict__ gu,
                                                              uint4* __restrict__ dgu, long long total, int iv) {
    const long long i = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (i >= total) return;
    const long long r = i / iv;
    const int c = (int)(i - r * iv);
    const uint4 dhv = ldg16(dh_act + i);
    const uint4 gv = ldg16(gu + r * (2 * iv) + c);
    const uint4 uv = ldg16(gu + r * (2 * iv) + iv + c);
    float dh[8], g[8], u[8], dg[8], du[8];
    unpack8(dhv, dh);
    unpack8(gv, g);
    unpack8(uv, u);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float s = 1.f / (1.f + __expf(-g[j]));
        dg[j] = dh[j] * u[j] * s * (1.f + g[j] * (1.f - s));
        du[j] = dh[j] * g[j] * s;
    }
    dgu[r * (2 * iv) + c] = pack8(dg);
    dgu[r * (2 * iv) + iv + c] = pack8(du);
}

inline unsigned blocks_for(long long total) { return (unsigned)((total + kThreads - 1) / kThreads); }

}  // namespace

size_t permute_workspace_bytes(const moe_dims_t& d) {
    const long long R = (long long)d.T * d.K;
    const long long n_chunks = (R + kWorkspacePairsPerRow - 1) / kWorkspacePairsPerRow;
    return (size_t)(n_chunks * d.E) * sizeof(int32_t);
}

// pairs per block-chunk: 2048, or more (a multiple of 256) when R is so large that the rank kernel's
// per-block sum over all histogram rows would otherwise grow past 512 rows
static int permute_chunk(long long R) {
    long long chunk = 2048;
    const long long need = (R + 511) / 512;
    if (need > chunk) chunk = (need + kThreads - 1) / kThreads * kThreads;
    return (int)chunk;
}

int movement_read_and_clear_status(int* status_out) {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_movement_status, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_movement_status, &zero, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    *status_out = v;
    return MOE_OK;
}

int launch_permute(const moe_dims_t& d, const bf16* x, const int32_t* topk_idx, bf16* x_perm, int32_t* counts,
                   int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row, void* workspace,
                   cudaStream_t s) {
    const int R = d.T * d.K, E = d.E;
    const int chunk = permute_chunk(R);
    const int n_blocks = (R + chunk - 1) / chunk;
    int32_t* ws = static_cast<int32_t*>(workspace);
    permute_hist_kernel<<<n_blocks, kThreads, E * sizeof(int32_t), s>>>(topk_idx, R, E, chunk, ws);
    // the two following kernels may start before their predecessor has finished (see grid_dependency_wait) -- for
    // small problems only, where the launch gaps are a third of the call; measured on the large ones (>= 131072
    // pairs) the early-started row kernel made the call 4-15 % slower
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    const unsigned n_pdl = R <= 65536 ? 1u : 0u;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_blocks); cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = ((kWarpsPerBlock + 3) * E + 1) * sizeof(int32_t); cfg.stream = s;
        cfg.attrs = pdl; cfg.numAttrs = n_pdl;
        const int32_t* ws_c = ws;
        if (cudaLaunchKernelEx(&cfg, permute_rank_kernel, topk_idx, R, E, chunk, n_blocks, ws_c, counts, offsets,
                               row_to_pair, pair_to_row) != cudaSuccess)
            return MOE_ERR_CUDA;
    }
    if (x_perm != nullptr) {
        const int row_bytes = d.H * 2;
        const int n_seg = (row_bytes + kRowMaxSeg - 1) / kRowMaxSeg;
        const int seg_bytes = ((row_bytes + n_seg - 1) / n_seg + 15) / 16 * 16;
        const size_t smem = (size_t)kRowBufs * seg_bytes;
        static bool attr_set[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
        if (!attr_set[dev]) {
            if (cudaFuncSetAttribute(permute_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kRowBufs * kRowMaxSeg) != cudaSuccess)
                return MOE_ERR_CUDA;
            attr_set[dev] = true;
        }
        const long long units = (long long)d.T * n_seg;
        const int per_sm = (int)(196608 / (smem + 1024) < 8 ? 196608 / (smem + 1024) : 8);
        long long grid = (long long)sm_count() * (per_sm < 1 ? 1 : per_sm);
        if (grid > units) grid = units;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(32); cfg.dynamicSmemBytes = smem; cfg.stream = s;
        cfg.attrs = pdl; cfg.numAttrs = n_pdl;
        const int32_t* p2r_c = pair_to_row;
        if (cudaLaunchKernelEx(&cfg, permute_rows_bulk_kernel, reinterpret_cast<const uint8_t*>(x), p2r_c,
                               reinterpret_cast<uint8_t*>(x_perm), d.T, d.K, row_bytes, seg_bytes, n_seg) != cudaSuccess)
            return MOE_ERR_CUDA;
    }
    return check_launch();
}

template <bool WEIGHTED>
static void gather_sum_dispatch(const moe_dims_t& d, const uint4* src, const float* w, const int32_t* p2r,
                                uint4* dst, cudaStream_t s) {
    const int hv = d.H / 8;
    const long long total = (long long)d.T * hv;
#define MOE_GS_CASE(KT)                                                                                          \
    case KT:                                                                                                     \
        gather_sum_kernel<KT, WEIGHTED><<<blocks_for(total), kThreads, 0, s>>>(src, w, p2r, dst, total, hv, d.K); \
        break;
    switch (d.K) {
        MOE_GS_CASE(1) MOE_GS_CASE(2) MOE_GS_CASE(3) MOE_GS_CASE(4) MOE_GS_CASE(5) MOE_GS_CASE(6) MOE_GS_CASE(7)
        MOE_GS_CASE(8)
        default:
            gather_sum_kernel<0, WEIGHTED><<<blocks_for(total), kThreads, 0, s>>>(src, w, p2r, dst, total, hv, d.K);
    }
#undef MOE_GS_CASE
}

int launch_gather_sum(const moe_dims_t& d, const bf16* src_perm, const float* topk_w, const int32_t* pair_to_row,
                      bf16* dst, cudaStream_t s) {
    const uint4* src = reinterpret_cast<const uint4*>(src_perm);
    uint4* out = reinterpret_cast<uint4*>(dst);
    if (topk_w != nullptr)
        gather_sum_dispatch<true>(d, src, topk_w, pair_to_row, out, s);
    else
        gather_sum_dispatch<false>(d, src, nullptr, pair_to_row, out, s);
    return check_launch();
}

template <bool WITH_DW>
static void combine_bwd_dispatch(const moe_dims_t& d, const uint4* dy, const uint4* yp, const float* w,
                                 const int32_t* p2r, uint4* dyp, float* dw, cudaStream_t s) {
    const int hv = d.H / 8;
    const unsigned blocks = (unsigned)d.T;
#define MOE_CB_CASE(KT)                                                                                     \
    case KT:                                                                                                \
        combine_bwd_kernel<KT, WITH_DW><<<blocks, kThreads, 0, s>>>(dy, yp, w, p2r, dyp, dw, d.T, hv, d.K); \
        break;
    switch (d.K) {
        MOE_CB_CASE(1) MOE_CB_CASE(2) MOE_CB_CASE(3) MOE_CB_CASE(4) MOE_CB_CASE(5) MOE_CB_CASE(6) MOE_CB_CASE(7)
        MOE_CB_CASE(8)
        default:
            combine_bwd_kernel<0, WITH_DW><<<blocks, kThreads, 0, s>>>(dy, yp, w, p2r, dyp, dw, d.T, hv, d.K);
    }
#undef MOE_CB_CASE
}

int launch_combine_bwd(const moe_dims_t& d, const bf16* dy, const bf16* y_perm, const float* topk_w,
                       const int32_t* pair_to_row, bf16* dy_perm, float* dtopk_w, cudaStream_t s) {
    const uint4* a = reinterpret_cast<const uint4*>(dy);
    const uint4* b = reinterpret_cast<const uint4*>(y_perm);
    uint4* o = reinterpret_cast<uint4*>(dy_perm);
    if (dtopk_w != nullptr)
        combine_bwd_dispatch<true>(d, a, b, topk_w, pair_to_row, o, dtopk_w, s);
    else
        combine_bwd_dispatch<false>(d, a, b, topk_w, pair_to_row, o, nullptr, s);
    return check_launch();
}

// ------------------------------------------------------------------------------------------------
// Route-permute without a caller-provided workspace.  The chunk-histogram table lives in a
// file-scope device array instead, so that a caller who may not allocate device memory (see the
// header) can still run the call.  The array's name is only a host-side handle in host code; the
// device address is looked up once per device with cudaGetSymbolAddress and handed to the
// ordinary permute launch.  Every entry the rank kernel reads is written by the histogram and
// scan kernels of the same call first, so nothing has to be cleared between calls.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_permute_static_scratch[MOE_PERMUTE_STATIC_SCRATCH_BYTES];

int launch_permute_static_scratch(const moe_dims_t& d, const bf16* x, const int32_t* topk_idx, bf16* x_perm,
                                  int32_t* counts, int32_t* offsets, int32_t* row_to_pair, int32_t* pair_to_row,
                                  cudaStream_t s) {
    if (permute_workspace_bytes(d) > (size_t)MOE_PERMUTE_STATIC_SCRATCH_BYTES) return MOE_ERR_WORKSPACE;
    static void* scratch_of_device[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    if (scratch_of_device[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_permute_static_scratch) != cudaSuccess || ptr == nullptr) return MOE_ERR_CUDA;
        scratch_of_device[dev] = ptr;
    }
    return launch_permute(d, x, topk_idx, x_perm, counts, offsets, row_to_pair, pair_to_row, scratch_of_device[dev], s);
}

int launch_swiglu_bwd(const moe_dims_t& d, const bf16* dh_act, const bf16* gu, bf16* dgu, cudaStream_t s) {
    const int iv = d.I / 8;
    const long long total = (long long)d.T * d.K * iv;
    swiglu_bwd_kernel<<<blocks_for(total), kThreads, 0, s>>>(reinterpret_cast<const uint4*>(dh_act),
                                                            reinterpret_cast<const uint4*>(gu),
                                                            reinterpret_cast<uint4*>(dgu), total, iv);
    return check_launch();
}

}  // namespace moe
