// Block-scaled FP8 (MXFP8) variant of the down projection: quantisers and a grouped GEMM on the block-scaled tensor-core
// path (tcgen05.mma kind::mxf8f6f4 with block_scale).
//
// Format: E4M3 elements, one E8M0 scale (a power of two, 2^(s-127)) per 32 consecutive elements along the
// contraction; scale of a block with largest magnitude a > 0: 2^(floor(log2 a) - 8); elements = v / scale rounded to
// nearest even, saturating at 448; an all-zero block: s = 0 and zero codes.  The decisions that produce integers
// (scale byte, element code) are taken on exact values on both sides of the parity test: the inputs are bf16, the
// division by a power of two is exact in fp32, and the FP8 conversion instruction rounds to nearest even.
//
// Layouts (chosen so that the GEMM's scale factors reach tensor memory without per-element work):
//   activation codes   [R, I] bytes, contraction contiguous
//   activation scales  [I/128][R] 32-bit words: the 4 scale bytes of the 4 blocks of 32 inside one 128-wide slice of
//                      the contraction, for one row -- rows of a tile start anywhere, so a warp gathers 128 words per
//                      K slice and lays them out for the tensor-memory copy
//   weight codes       [E, H, I] bytes: the down weights transposed, contraction contiguous
//   weight scales      [E][H/128][I/128][512 bytes]: per 128 output features x 128 contraction elements, byte
//                      (h % 32) * 16 + ((h % 128) / 32) * 4 + block -- the 32 x 16-byte pattern that
//                      tcgen05.cp.32x128b.warpx4 copies from shared memory into 4 tensor-memory columns (lane = h % 32,
//                      column = (h % 128) / 32, byte = block)
//
// GEMM kernel: one CTA per SM, persistent over the same row-ragged tile list as the bf16 kernels (tiles of 128 rows x
// 128 output features), K slices of 128 (= 128 bytes per row: the same swizzled stage geometry as 64 bf16).
//   warp 0      TMA producer: A and B code tiles, bulk copy of the weight-scale block
//   warp 1      one thread: tcgen05.cp of both scale blocks into tensor memory, four tcgen05.mma (K = 32 each, scale
//               byte k selected through the instruction descriptor), commit
//   warp 2      activation scales: gathers the tile's 128 words of the K slice and writes them in the copy's pattern
//   warps 3..6  epilogue: tcgen05.ld, round to bf16, staged bulk tensor stores
// Accumulator double buffered (2 x 128 columns); the scale blocks of a stage use 8 tensor-memory columns, two such
// slots alternate (copies and MMAs of one thread execute in issue order).
#include <cuda_fp8.h>

#include "tc_ptx.cuh"

namespace moe {

__device__ int g_mx_status = 0;

int mx_read_and_clear_status(int* status_out) {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_mx_status, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_mx_status, &zero, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    *status_out = v;
    return MOE_OK;
}

namespace {

constexpr int MX_BM = 128, MX_BN = 128, MX_BK = 128;   // tile rows, tile columns, contraction elements per stage
constexpr int MX_STAGES = 6;
constexpr int MX_A_BYTES = MX_BM * MX_BK, MX_B_BYTES = MX_BN * MX_BK, MX_SF_BYTES = 512;
constexpr int MX_STAGE_BYTES = MX_A_BYTES + MX_B_BYTES + 2 * MX_SF_BYTES;   // 33 KB
constexpr int MX_EPI_WARPS = 4;
constexpr int MX_THREADS = 32 * (3 + MX_EPI_WARPS);
constexpr int MX_STAGING_BYTES = MX_EPI_WARPS * 2048;
constexpr int MX_MAX_E = 1024;
constexpr int MX_TMEM_COLS = 512;
constexpr int MX_SF_COL0 = 2 * MX_BN;   // first tensor-memory column of the scale slots (after the two accumulators)

struct MxCtl {
    unsigned long long full[MX_STAGES];
    unsigned long long empty[MX_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    uint32_t tmem_base;
    int abort_flag;
    int32_t offs[MX_MAX_E + 1];
    int32_t tile_prefix[MX_MAX_E + 1];
};
constexpr int MX_SMEM_BYTES = MX_STAGES * MX_STAGE_BYTES + MX_STAGING_BYTES + 1024 + (int)sizeof(MxCtl);
static_assert(MX_SMEM_BYTES <= 232448, "exceeds the shared memory a CTA can opt in to");

struct MxParams {
    const int32_t* offsets;
    int E, k_tiles, n_tiles, n_cols;
    long long R;
    const uint32_t* sa;   // activation scale words [k_tiles][R]
    const uint8_t* sb;    // weight scale blocks [E][n_tiles][k_tiles][512]
    bf16* out;
    long long ldo;
};

__device__ __forceinline__ bool mx_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return mbar_wait_status(bar, parity, abort_flag, &g_mx_status);
}

// K-major operand tile [rows][128 bytes], 128-byte swizzle: 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t mx_operand_desc(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Scale block [32 rows][16 bytes], no swizzle: 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t mx_scale_desc(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(128 >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor of the block-scaled kind: E4M3 x E4M3, both K-major, E8M0 scales, scale byte `sf` of the
// scale columns for both operands.
__device__ __forceinline__ uint32_t mx_idesc(uint32_t sf) {
    return (sf << 4) | ((uint32_t)(MX_BN >> 3) << 17) | (1u << 23) | ((uint32_t)(MX_BM >> 4) << 24) | (sf << 29);
}
__device__ __forceinline__ void mx_copy_scales(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void mx_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa,
                                       uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.u32 p, %4, 0;"
        " tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p; }" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
}

struct MxTile {
    int e, row0, row_end, n0;
};
__device__ __forceinline__ MxTile mx_decode(const MxParams& p, const MxCtl* ctl, long long t) {
    int lo = 0, hi = p.E;   // largest e with tile_prefix[e] * n_tiles <= t
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)ctl->tile_prefix[mid] * p.n_tiles <= t) lo = mid; else hi = mid;
    }
    const int local = (int)(t - (long long)ctl->tile_prefix[lo] * p.n_tiles);
    const int m_tiles_e = ctl->tile_prefix[lo + 1] - ctl->tile_prefix[lo];
    MxTile tl;
    tl.e = lo;
    // column tile major inside an expert: the CTAs that run at the same time share the expert's weight tiles in L2
    const int nt = local / m_tiles_e, mt = local - nt * m_tiles_e;
    tl.row0 = ctl->offs[lo] + mt * MX_BM;
    tl.row_end = ctl->offs[lo + 1];
    tl.n0 = nt * MX_BN;
    return tl;
}

__global__ void __launch_bounds__(MX_THREADS, 1)
mx_down_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_o, const MxParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
    MxCtl* ctl = reinterpret_cast<MxCtl*>(tiles_ptr + MX_STAGES * MX_STAGE_BYTES + MX_STAGING_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int e = threadIdx.x; e <= p.E; e += MX_THREADS) ctl->offs[e] = p.offsets[e];
    if (threadIdx.x == 0) {
        for (int s = 0; s < MX_STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2);    // the producer's arrive (with the byte count) + the scale warp's
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctl->tmem_full[a]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[a]), MX_EPI_WARPS);
        }
        mbar_init(smem_u32(&ctl->drain), 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
        prefetch_tmap(&map_o);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < p.E; ++e) {
            ctl->tile_prefix[e] = run;
            run += (ctl->offs[e + 1] - ctl->offs[e] + MX_BM - 1) / MX_BM;
        }
        ctl->tile_prefix[p.E] = run;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"((uint32_t)MX_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const long long n_tiles_total = (long long)ctl->tile_prefix[p.E] * p.n_tiles;
    auto stage_base = [&](uint32_t s) { return tiles_base + s * MX_STAGE_BYTES; };

    if (warp == 0) {
        // ================= producer =================
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < n_tiles_total; t += gridDim.x) {
                const MxTile tl = mx_decode(p, ctl, t);
                const uint8_t* sb_tile = p.sb + ((long long)tl.e * p.n_tiles + tl.n0 / MX_BN) * p.k_tiles * MX_SF_BYTES;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    if (!mx_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t a_dst = stage_base(stage);
                    mbar_arrive_expect_tx(full, MX_A_BYTES + MX_B_BYTES + MX_SF_BYTES);
                    tma_load_2d(a_dst, &map_a, kt * MX_BK, tl.row0, full);
                    tma_load_2d(a_dst + MX_A_BYTES, &map_b, kt * MX_BK, tl.e * p.n_cols + tl.n0, full);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                                     a_dst + MX_A_BYTES + MX_B_BYTES + MX_SF_BYTES),
                                 "l"(sb_tile + (long long)kt * MX_SF_BYTES), "r"(MX_SF_BYTES), "r"(full)
                                 : "memory");
                    ++issued;
                    if (++stage == MX_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {   // leave no bulk copy in flight: bounded wait for the copies issued into each stage
                const uint32_t n_wait = issued < (uint32_t)MX_STAGES ? issued : (uint32_t)MX_STAGES;
                uint32_t s = stage, ph = phase;
                for (uint32_t i = 0; i < n_wait; ++i) {
                    if (s == 0) { s = MX_STAGES - 1; ph ^= 1u; } else { --s; }
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(smem_u32(&ctl->full[s]), ph) && global_timer_ns() - t0 < WAIT_LIMIT_NS / 4) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer: one thread =================
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0, slot = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < n_tiles_total; t += gridDim.x) {
                if (!mx_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * MX_BN;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    if (!mx_wait(smem_u32(&ctl->full[stage]), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = stage_base(stage);
                    const uint32_t sfa_t = tmem_base + MX_SF_COL0 + slot * 8, sfb_t = sfa_t + 4;
                    mx_copy_scales(sfa_t, mx_scale_desc(a_base + MX_A_BYTES + MX_B_BYTES));
                    mx_copy_scales(sfb_t, mx_scale_desc(a_base + MX_A_BYTES + MX_B_BYTES + MX_SF_BYTES));
                    const uint64_t a_desc = mx_operand_desc(a_base), b_desc = mx_operand_desc(a_base + MX_A_BYTES);
#pragma unroll
                    for (int k = 0; k < MX_BK / 32; ++k)
                        mx_mma(d_tmem, a_desc + (uint64_t)((k * 32) >> 4), b_desc + (uint64_t)((k * 32) >> 4), mx_idesc(k), sfa_t,
                               sfb_t, (kt != 0 || k != 0) ? 1u : 0u);
                    tc_commit<false>(smem_u32(&ctl->empty[stage]));
                    slot ^= 1u;
                    if (++stage == MX_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit<false>(smem_u32(&ctl->tmem_full[acc]));
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            // all issued copies and MMAs must have retired before tensor memory is released
            tc_commit_local<false>(smem_u32(&ctl->drain));
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < WAIT_LIMIT_NS) {}
        }
        __syncwarp();
    } else if (warp == 2) {
        // ================= activation scales =================
        // lane l owns rows l, 32 + l, 64 + l, 96 + l of the tile: one 16-byte piece of the 32 x 16-byte block
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (long long t = blockIdx.x; ok && t < n_tiles_total; t += gridDim.x) {
            const MxTile tl = mx_decode(p, ctl, t);
            long long rows[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const long long r = (long long)tl.row0 + 32 * i + lane;
                rows[i] = r < p.R ? r : p.R - 1;   // rows past the end are never stored; any valid address will do
            }
            uint4 next;
            next.x = __ldg(p.sa + rows[0]); next.y = __ldg(p.sa + rows[1]); next.z = __ldg(p.sa + rows[2]); next.w = __ldg(p.sa + rows[3]);
            for (int kt = 0; kt < p.k_tiles; ++kt) {
                const uint4 cur = next;
                if (kt + 1 < p.k_tiles) {   // the next slice's words travel while this one waits for its stage
                    const uint32_t* s = p.sa + (long long)(kt + 1) * p.R;
                    next.x = __ldg(s + rows[0]); next.y = __ldg(s + rows[1]); next.z = __ldg(s + rows[2]); next.w = __ldg(s + rows[3]);
                }
                if (!mx_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
                *reinterpret_cast<uint4*>(tiles_ptr + stage * MX_STAGE_BYTES + MX_A_BYTES + MX_B_BYTES + lane * 16) = cur;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->full[stage]));
                if (++stage == MX_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else {
        // ================= epilogue (warps 3..6) =================
        const int quarter = warp & 3;   // tensor-memory lanes [32 * quarter, 32 * quarter + 32)
        uint8_t* stage_ptr = tiles_ptr + MX_STAGES * MX_STAGE_BYTES + (warp - 3) * 2048;
        const int sw = (lane >> 1) & 3;
        uint32_t n_stores = 0, acc = 0, acc_phase = 0;
        for (long long t = blockIdx.x; t < n_tiles_total; t += gridDim.x) {
            const MxTile tl = mx_decode(p, ctl, t);
            if (!mx_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + acc * MX_BN + ((uint32_t)(quarter * 32) << 16);
            const int slab0 = tl.row0 + quarter * 32;
            const int rows_valid = max(0, min(32, tl.row_end - slab0));
#pragma unroll 1
            for (int c = 0; c < MX_BN / 32; ++c) {
                uint32_t v[32];
                tc_ld32(taddr + c * 32, v);
                tc_wait_ld();
                const int n = tl.n0 + c * 32;
                if (rows_valid == 0 || n >= p.n_cols) continue;
                uint32_t w[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) w[j] = pack_bf16(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                if (rows_valid == 32) {
                    if (n_stores != 0) {
                        if (lane == 0) bulk_wait_read0();
                        __syncwarp();
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(stage_ptr + lane * 64 + ((j ^ sw) << 4)) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&map_o, n, slab0, smem_u32(stage_ptr));
                        bulk_commit();
                    }
                    ++n_stores;
                } else if (lane < rows_valid) {
                    uint4* d4 = reinterpret_cast<uint4*>(p.out + ((long long)slab0 + lane) * p.ldo + n);
#pragma unroll
                    for (int j = 0; j < 4; ++j) d4[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (n_stores != 0 && lane == 0) bulk_wait_all0();
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)MX_TMEM_COLS) : "memory");
    }
}

// ---- quantisers ---------------------------------------------------------------------------------------
// scale exponent of a block with largest magnitude amax: floor(log2 amax) - 8, clamped to the E8M0 range; -127 for zero
__device__ __forceinline__ int mx_scale_exp(float amax) {
    if (!(amax > 0.f)) return -127;
    const int e = ilogbf(amax) - 8;
    return e < -127 ? -127 : (e > 127 ? 127 : e);
}
// 2^-s as a float (s in [-127, 127]; 2^-127 is a subnormal)
__device__ __forceinline__ float mx_inv_scale(int s) {
    return s == 127 ? __int_as_float(0x00400000) : __int_as_float((127 - s) << 23);
}
__device__ __forceinline__ uint32_t mx_e4m3(float v) {
    return (uint32_t)__nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
}

// rows x n bf16 -> codes and scale words.  One warp per (row, 128-wide slice): lane l holds elements 4l..4l+3, the 8
// lanes of a block of 32 agree on its scale through three shuffles.
__global__ void __launch_bounds__(256) mx_quantize_rows_kernel(const uint2* __restrict__ x, long long rows, int n,
                                                               uint32_t* __restrict__ codes, uint32_t* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const int k_tiles = n / 128;
    for (long long u = warp; u < rows * k_tiles; u += n_warps) {
        const long long r = u / k_tiles;
        const int kt = (int)(u - r * k_tiles);
        const uint2 raw = __ldg(x + (r * n + kt * 128) / 4 + lane);
        const float2 v01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 v23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        float amax = fmaxf(fmaxf(fabsf(v01.x), fabsf(v01.y)), fmaxf(fabsf(v23.x), fabsf(v23.y)));
#pragma unroll
        for (int s = 1; s < 8; s <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, s));
        const int se = mx_scale_exp(amax);
        const float inv = mx_inv_scale(se);
        codes[(r * n + kt * 128) / 4 + lane] = mx_e4m3(v01.x * inv) | (mx_e4m3(v01.y * inv) << 8) | (mx_e4m3(v23.x * inv) << 16) |
                                               (mx_e4m3(v23.y * inv) << 24);
        const uint32_t sbyte = (uint32_t)(se + 127);
        const uint32_t word = __shfl_sync(0xffffffffu, sbyte, 0) | (__shfl_sync(0xffffffffu, sbyte, 8) << 8) |
                              (__shfl_sync(0xffffffffu, sbyte, 16) << 16) | (__shfl_sync(0xffffffffu, sbyte, 24) << 24);
        if (lane == 0) scales[(long long)kt * rows + r] = word;
    }
}

// w_down [E, I, H] bf16 -> codes [E, H, I] and scale blocks.  One thread per (expert, block of 32 along I, feature h):
// consecutive lanes take consecutive h, so the 32 loads of a thread are coalesced across the warp; the thread keeps the
// 32 values, picks the scale and writes 32 contiguous code bytes.
__global__ void __launch_bounds__(256) mx_quantize_w_down_kernel(const bf16* __restrict__ w, int E, int I, int H,
                                                                 uint8_t* __restrict__ codes, uint8_t* __restrict__ scales) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int blocks_i = I / 32;
    const long long total = (long long)E * blocks_i * H;
    if (idx >= total) return;
    const int h = (int)(idx % H);
    const int ib = (int)((idx / H) % blocks_i);
    const int e = (int)(idx / ((long long)H * blocks_i));
    const bf16* src = w + ((long long)e * I + (long long)ib * 32) * H + h;
    float v[32];
    float amax = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        v[j] = __bfloat162float(src[(long long)j * H]);
        amax = fmaxf(amax, fabsf(v[j]));
    }
    const int se = mx_scale_exp(amax);
    const float inv = mx_inv_scale(se);
    uint32_t out[8];
#pragma unroll
    for (int q = 0; q < 8; ++q)
        out[q] = mx_e4m3(v[4 * q] * inv) | (mx_e4m3(v[4 * q + 1] * inv) << 8) | (mx_e4m3(v[4 * q + 2] * inv) << 16) |
                 (mx_e4m3(v[4 * q + 3] * inv) << 24);
    uint4* dst = reinterpret_cast<uint4*>(codes + ((long long)e * H + h) * I + (long long)ib * 32);
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
    const int k_tiles = I / 128;
    scales[(((long long)e * (H / 128) + h / 128) * k_tiles + ib / 4) * 512 + (h % 32) * 16 + ((h % 128) / 32) * 4 + (ib % 4)] =
        (uint8_t)(se + 127);
}

}  // namespace

int launch_mx_quantize_rows(long long rows, int n, const bf16* x, uint8_t* codes, uint8_t* scales, cudaStream_t s) {
    const long long units = rows * (n / 128);
    long long blocks = (units + 7) / 8;
    const long long cap = (long long)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    mx_quantize_rows_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const uint2*>(x), rows, n,
                                                           reinterpret_cast<uint32_t*>(codes), reinterpret_cast<uint32_t*>(scales));
    return check_launch();
}

int launch_mx_quantize_w_down(const moe_dims_t& d, const bf16* w_down, uint8_t* codes_t, uint8_t* scales, cudaStream_t s) {
    const long long total = (long long)d.E * (d.I / 32) * d.H;
    mx_quantize_w_down_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(w_down, d.E, d.I, d.H, codes_t, scales);
    return check_launch();
}

int launch_down_fwd_mxfp8(const moe_dims_t& d, const uint8_t* h_codes, const uint8_t* h_scales, const uint8_t* w_codes_t,
                          const uint8_t* w_scales, const int32_t* offsets, bf16* y_perm, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    CUtensorMap a, b, o;
    if (!make_map_typed(&a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, h_codes, d.I, R, MX_BK, MX_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w_codes_t, d.I, (uint64_t)d.E * d.H, MX_BK, MX_BN,
                        CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_out_map(&o, y_perm, d.H, R))
        return MOE_ERR_CUDA;
    MxParams p = {};
    p.offsets = offsets; p.E = d.E; p.k_tiles = d.I / MX_BK; p.n_tiles = d.H / MX_BN; p.n_cols = d.H; p.R = (long long)R;
    p.sa = reinterpret_cast<const uint32_t*>(h_scales); p.sb = w_scales; p.out = y_perm; p.ldo = d.H;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(mx_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MX_SMEM_BYTES) != cudaSuccess)
            return MOE_ERR_CUDA;
        attr_set[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return MOE_ERR_CUDA;
    mx_down_kernel<<<sms, MX_THREADS, MX_SMEM_BYTES, s>>>(a, b, o, p);
    return check_launch();
}

}  // namespace moe
