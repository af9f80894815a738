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
// a1 in two launches.
//   hist      : one block per `chunk` consecutive pairs (a multiple of 256): the number of pairs of each
//               expert in the chunk (shared-memory atomics: counts are order-free)          -> ws[chunk][e]
//   rank_rows : one block per kTokPerBlock consecutive tokens.  The block
//               (1) starts bulk loads of its first token rows and counts, from the routing indices alone,
//                   the pairs between the start of its histogram chunk and its own first pair, and its own
//                   pairs per warp -- all before the histogram kernel's output is needed;
//               (2) sums the histogram rows: all of them (the counts), those before its chunk (its base);
//                   counts -> offsets by a warp scan;
//               (3) ranks its own pairs: row(p) = offsets[e] + base[e] + pairs of e in earlier warps of
//                   the block + earlier pairs of e in the same warp (same-expert lane mask of each 32
//                   pairs from 32 broadcasts, and popc): the unique stable sort, no atomic decides an index;
//               (4) pushes its tokens' rows to their K destination rows with the bulk-copy engine: a ring
//                   of shared-memory buffers, one cp.async.bulk load per row (or <= 16 KB segment), K
//                   cp.async.bulk stores (lane k issues store k).  Each row is read from HBM once, no data
//                   passes through registers, and a block copies as soon as ITS pairs are ranked: nothing
//                   waits for the whole index to exist.
// A pair whose expert id lies outside [0, E) is dropped (it gets no row; the rows past offsets[E] stay
// unwritten) and MOE_ERR_BAD_INDEX is recorded in the device status word.
// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch: rank_rows may start (and run step 1) while hist is still finishing;
// grid_dependency_wait() then blocks until everything hist wrote is visible.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr int kIdxGroup = 8;   // index loads in flight per thread in the permute index kernels
__device__ int g_movement_status = 0;

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

// Geometry of rank_rows, from sweeps on B200 over the benchmark workloads (whole call, L2 flushed): 8 warps, 4
// tokens per block and a ring of 3 buffers with loads 2 units ahead were best everywhere.  Blocks this small keep
// eight of them resident per SM, each in a different phase (counting, ranking, copying); larger blocks, deeper rings
// or 4-warp blocks (more but slower blocks per SM) all lost 5-20 % on the large workloads.
constexpr int kPermWarps = 8, kPermThreads = 32 * kPermWarps;
constexpr int kTokPerBlock = 4;
constexpr int kRowBufs = 3, kRowLookahead = 2, kRowMaxSeg = 16384;
constexpr int kMaxOwnPairs = kTokPerBlock * 32;   // K <= 32
static_assert(kMaxOwnPairs <= 32 * kPermWarps, "each warp ranks at most one group of 32 own pairs");
constexpr unsigned long long kRowWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long movement_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for a bulk load (2 s on %globaltimer).  False when the wait ran out.
__device__ __forceinline__ bool row_bar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        uint32_t done;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done)
                     : "r"(bar), "r"(parity)
                     : "memory");
        if (done) return true;
        if ((spin & 0xFF) == 0xFF) {
            const unsigned long long now = movement_timer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) return false;
        }
    }
}

// Shared memory of rank_rows: the row ring first (128-byte aligned), then the index tables.
struct RankRowsSmem {
    int ring_bytes;     // kRowBufs * seg_bytes, 0 without a row copy
    int total_bytes;
    __host__ __device__ RankRowsSmem(int E, int seg_bytes, bool rows) {
        ring_bytes = rows ? kRowBufs * seg_bytes : 0;
        total_bytes = ring_bytes + ((kPermWarps + 3) * E + 1 + kMaxOwnPairs) * (int)sizeof(int32_t);
    }
};

__global__ void __launch_bounds__(kPermThreads) permute_rank_rows_kernel(
    const int32_t* __restrict__ topk_idx, int R, int E, int K, int T, int chunk, int n_chunks,
    const int32_t* __restrict__ ws, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
    int32_t* __restrict__ row_to_pair, int32_t* __restrict__ pair_to_row, const uint8_t* __restrict__ x,
    uint8_t* __restrict__ x_perm, int row_bytes, int seg_bytes, int n_seg) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ unsigned long long bars[kRowBufs];
    const bool rows = x_perm != nullptr;
    const RankRowsSmem lay(E, seg_bytes, rows);
    uint8_t* bufs = smem_raw;                                        // [kRowBufs][seg_bytes]
    int32_t* offs = reinterpret_cast<int32_t*>(smem_raw + lay.ring_bytes);   // [E+1] exclusive prefix of the counts
    int32_t* total = offs + (E + 1);                                 // [E]   counts
    int32_t* base = total + E;                                       // [E]   pairs of e before this block's first pair
    int32_t* whist = base + E;                                       // [warps][E] per-warp counts, then running row cursors
    int32_t* dest = whist + kPermWarps * E;                      // [own pairs] destination row of each own pair (-1: dropped)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int t0 = blockIdx.x * kTokPerBlock, t1 = min(T, t0 + kTokPerBlock);
    const long long p_begin = (long long)t0 * K, p_end = (long long)t1 * K;
    const int n_own = (int)(p_end - p_begin);
    const int my_chunk = (int)(p_begin / chunk);                     // histogram rows wholly before this block: a < my_chunk
    const long long chunk_begin = (long long)my_chunk * chunk;
    const int n_units = rows ? (t1 - t0) * n_seg : 0;                // row segments this block copies
    const int n_pre = min(kRowLookahead, n_units);

    // ---- (1) nothing here needs the histogram kernel's output ----
    auto issue_load = [&](int u) {   // lane 0 of warp 0
        const int s = u % kRowBufs;
        const int t = t0 + u / n_seg, seg = u % n_seg;
        const int bytes = min(seg_bytes, row_bytes - seg * seg_bytes);
        const uint32_t bar = smem_addr(&bars[s]);
        asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_addr(bufs + (size_t)s * seg_bytes)),
                     "l"(x + (long long)t * row_bytes + (long long)seg * seg_bytes), "r"(bytes), "r"(bar)
                     : "memory");
    };
    if (threadIdx.x == 0 && rows) {
        for (int s = 0; s < kRowBufs; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[s])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int u = 0; u < n_pre; ++u) issue_load(u);
    }
    // this warp's contiguous share of the block's own pairs (at most 32: one per lane); the expert id stays in a
    // register from here to the ranking pass.  -1: no pair here; -2: a pair with an invalid expert id
    const int per_warp = (n_own + kPermWarps - 1) / kPermWarps;
    const long long my_p = p_begin + (long long)warp * per_warp + lane;
    int own = -1;
    bool bad = false;
    if (lane < per_warp && my_p < p_end) {
        own = topk_idx[my_p];
        if (own < 0 || own >= E) { bad = true; own = -2; }
    }
    // pairs between the start of the histogram chunk and this block's first pair (fewer than `chunk`): the first
    // batch of their ids is requested before anything waits
    const int n_before = (int)(p_begin - chunk_begin);
    int before0[kIdxGroup];
#pragma unroll
    for (int g = 0; g < kIdxGroup; ++g) {
        const int i = (int)threadIdx.x + g * kPermThreads;
        before0[g] = i < n_before ? topk_idx[chunk_begin + i] : -1;
    }
    for (int i = threadIdx.x; i < (kPermWarps + 2) * E; i += kPermThreads) total[i] = 0;   // total, base, whist
    __syncthreads();
#pragma unroll
    for (int g = 0; g < kIdxGroup; ++g)
        if (before0[g] >= 0 && before0[g] < E) atomicAdd(&base[before0[g]], 1);   // counts only: order-free
    for (int i0 = threadIdx.x + kPermThreads * kIdxGroup; i0 < n_before; i0 += kPermThreads * kIdxGroup) {
        int ev[kIdxGroup];
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g) {
            const int i = i0 + g * kPermThreads;
            ev[g] = i < n_before ? topk_idx[chunk_begin + i] : -1;
        }
#pragma unroll
        for (int g = 0; g < kIdxGroup; ++g)
            if (ev[g] >= 0 && ev[g] < E) atomicAdd(&base[ev[g]], 1);
    }
    // pass 1: this warp's histogram over its own pairs
    int32_t* mine = whist + warp * E;
    if (own >= 0) atomicAdd(&mine[own], 1);   // counts only: order-free
    // ---- (2) the chunk histograms are complete and visible from here on ----
    grid_dependency_wait();
    for (int i = threadIdx.x; i < n_chunks * E; i += kPermThreads) {
        const int v = ws[i];
        if (v != 0) {
            const int a = i / E, e = i - a * E;
            atomicAdd(&total[e], v);
            if (a < my_chunk) atomicAdd(&base[e], v);
        }
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
        for (int e = threadIdx.x; e <= E; e += kPermThreads) offsets[e] = offs[e];
        for (int e = threadIdx.x; e < E; e += kPermThreads) counts[e] = total[e];
    }
    // per-warp counts -> first row of each (warp, expert)
    for (int e = threadIdx.x; e < E; e += kPermThreads) {
        int run = offs[e] + base[e];
#pragma unroll
        for (int w = 0; w < kPermWarps; ++w) {
            const int v = whist[w * E + e];
            whist[w * E + e] = run;
            run += v;
        }
    }
    __syncthreads();
    // ---- (3) stable ranks of the own pairs ----
    {
        // lanes of the warp with the same expert: 32 broadcasts are several times faster than match.any here
        // (whose time grows with the number of distinct values, and routing makes most of them distinct)
        unsigned mask = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) mask |= (__shfl_sync(0xffffffffu, own, j) == own ? 1u : 0u) << j;
        if (own >= 0) {
            const int row = mine[own] + __popc(mask & ((1u << lane) - 1u));
            row_to_pair[row] = (int32_t)my_p;
            pair_to_row[my_p] = row;
            dest[my_p - p_begin] = row;
        } else if (own == -2) {
            dest[my_p - p_begin] = -1;
        }
    }
    if (bad) atomicExch(&g_movement_status, (int)MOE_ERR_BAD_INDEX);
    __syncthreads();
    // ---- (4) rows: warp 0 runs the ring, loads kRowLookahead units ahead of the stores ----
    if (warp != 0 || n_units == 0) return;
    bool ok = true;
    int loads_issued = n_pre;
    for (int it = 0; it < n_units + kRowLookahead; ++it) {
        if (it >= n_pre && it < n_units) {
            // the stores that last read this buffer were committed kRowBufs - kRowLookahead iterations ago
            if (it >= kRowBufs) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kRowBufs - kRowLookahead - 1) : "memory");
            __syncwarp();
            if (lane == 0) issue_load(it);
            loads_issued = it + 1;
        }
        const int j = it - kRowLookahead;
        if (j >= 0) {
            const int s = j % kRowBufs;
            const uint32_t parity = (uint32_t)((j / kRowBufs) & 1);
            const int t = t0 + j / n_seg, seg = j % n_seg;
            const int bytes = min(seg_bytes, row_bytes - seg * seg_bytes);
            ok = row_bar_wait(smem_addr(&bars[s]), parity, kRowWaitLimitNs);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                // give up: report, and leave no load in flight (bounded wait for each load issued after this one)
                if (lane == 0) atomicExch(&g_movement_status, (int)MOE_ERR_TIMEOUT);
                for (int u = j + 1; u < loads_issued; ++u)
                    row_bar_wait(smem_addr(&bars[u % kRowBufs]), (uint32_t)((u / kRowBufs) & 1), kRowWaitLimitNs / 8);
                break;
            }
            const int row = lane < K ? dest[(t - t0) * K + lane] : -1;
            if (row >= 0) {
                uint8_t* dst = x_perm + (long long)row * row_bytes + (long long)seg * seg_bytes;
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
// (three blocks per SM: with the 80 registers that allows nothing spills; at five blocks per SM the K = 8 kernel
// spilled and ran 16 % slower inside a step; the instance for a run-time K keeps 32 accumulators and takes two blocks).
// ------------------------------------------------------------------------------------------------
template <int KT, bool WITH_DW>
__global__ void __launch_bounds__(kThreads, KT > 0 ? 3 : 2) combine_bwd_kernel(const uint4* __restrict__ dy,
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
        // approximate division (2 ulp): inside a power-capped step this kernel is bound by instruction issue at the
        // low clock, not by HBM -- the exact division cost 18 % of its time there
        const float s = __fdividef(1.f, 1.f + __expf(-g[j]));
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

// pairs per histogram chunk: 2048, or more (a multiple of 256) when R is so large that the sum over all
// histogram rows in every rank_rows block would otherwise grow past 512 rows
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
    const int n_chunks = (R + chunk - 1) / chunk;
    int32_t* ws = static_cast<int32_t*>(workspace);
    permute_hist_kernel<<<n_chunks, kThreads, E * sizeof(int32_t), s>>>(topk_idx, R, E, chunk, ws);

    const bool rows = x_perm != nullptr;
    const int row_bytes = d.H * 2;
    const int n_seg = (row_bytes + kRowMaxSeg - 1) / kRowMaxSeg;
    const int seg_bytes = ((row_bytes + n_seg - 1) / n_seg + 15) / 16 * 16;
    const RankRowsSmem lay(E, seg_bytes, rows);
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    if (!attr_set[dev]) {
        const RankRowsSmem largest(1024, kRowMaxSeg, true);
        if (cudaFuncSetAttribute(permute_rank_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 largest.total_bytes) != cudaSuccess)
            return MOE_ERR_CUDA;
        attr_set[dev] = true;
    }
    const unsigned grid = (unsigned)((d.T + kTokPerBlock - 1) / kTokPerBlock);
    // launched as a programmatic dependent of the histogram kernel: its blocks start, prefetch rows and count from
    // the routing indices while the histogram kernel is still running
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kPermThreads); cfg.dynamicSmemBytes = lay.total_bytes; cfg.stream = s;
    cfg.attrs = pdl; cfg.numAttrs = 1;
    const int32_t* ws_c = ws;
    if (cudaLaunchKernelEx(&cfg, permute_rank_rows_kernel, topk_idx, R, E, (int)d.K, (int)d.T, chunk,
                           n_chunks, ws_c, counts, offsets, row_to_pair, pair_to_row,
                           reinterpret_cast<const uint8_t*>(x), reinterpret_cast<uint8_t*>(x_perm), row_bytes,
                           seg_bytes, n_seg) != cudaSuccess)
        return MOE_ERR_CUDA;
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
// ordinary permute launch.  Every entry the second kernel reads is written by the histogram kernel of
// the same call first, so nothing has to be cleared between calls.
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
