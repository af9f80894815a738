// Block-scaled FP8 (MXFP8) twins of the six grouped GEMMs (gate/up forward, down forward, down dgrad, gate/up dgrad, and
// the two weight gradients, further down) on the block-scaled tensor-core path (tcgen05.mma kind::mxf8f6f4 with block_scale): quantisers, one GEMM
// in two tilings, and the SwiGLU activation with the activation quantiser fused in.  Every GEMM here is
//   out[r, :] = dequant(a row r) . dequant(b[e])^T   for the rows r of expert e,
// a [R, k] and b [E, n_feat, k] both contraction-contiguous; the callers choose which tensors play a and b.
//
// Format: E4M3 elements, one E8M0 scale (a power of two, 2^(s-127)) per 32 consecutive elements along the
// contraction; scale of a block with largest magnitude a > 0: 2^(floor(log2 a) - 8); elements = v / scale rounded to
// nearest even, saturating at 448; an all-zero block: s = 0 and zero codes.  The decisions that produce integers
// (scale byte, element code) are taken on exact values on both sides of the parity test: the inputs are bf16, the
// division by a power of two is exact in fp32, and the FP8 conversion instruction rounds to nearest even.
//
// Layouts (chosen so that the GEMM's scale factors reach tensor memory without per-element work):
//   activation codes   [R, k] bytes, contraction contiguous
//   activation scales  [k/128][R] 32-bit words: the 4 scale bytes of the 4 blocks of 32 inside one 128-wide slice of
//                      the contraction, for one row -- rows of a tile start anywhere, so a warp gathers 128 words per
//                      K slice and lays them out for the tensor-memory copy
//   weight codes       [E, n_feat, k] bytes, contraction contiguous (weights stored feature-contiguous are transposed by
//                      their quantiser)
//   weight scales      first [E][n_feat/128][k/128][512 bytes]: per 128 output features x 128 contraction elements, byte
//                      (f % 32) * 16 + ((f % 128) / 32) * 4 + block -- the 32 x 16-byte pattern that
//                      tcgen05.cp.32x128b.warpx4 copies from shared memory into 4 tensor-memory columns (lane = f % 32,
//                      column = (f % 128) / 32, byte = block); then the same bytes in the tiling of the CTA-pair kernel
//                      (see there)
//
// Single-CTA kernel: one CTA per SM, persistent over the same row-ragged tile list as the bf16 kernels (tiles of 128 rows x
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

#ifdef MOE_TEST_HOOKS
// Test-only build: when set, every producer leaves out the loads and the barrier arrival of its first ring stage, so that
// the bounded waits on that stage run out (see grouped_gemm.cu).
__device__ int g_mx_test_withhold_first_stage = 0;
extern "C" int moe_test_withhold_first_stage_mxfp8(int on) {
    return cudaMemcpyToSymbol(g_mx_test_withhold_first_stage, &on, sizeof(int)) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
#endif

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
constexpr int MX_SCALE_AHEAD = 4;   // K slices whose activation-scale words the scale warp keeps in flight
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

// (roles in which a whole warp waits take the verdict through __all_sync: a wait that runs out for one lane while the
// barrier completes for another must not split the warp ahead of a warp-wide instruction)
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
mx_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
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
#ifdef MOE_TEST_HOOKS
                    if (g_mx_test_withhold_first_stage != 0 && issued == 0) {
                        ++issued;
                        if (++stage == MX_STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
#endif
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
            // the words of MX_SCALE_AHEAD slices are in flight at any time: one slice per global-load round trip would
            // bound the whole pipeline (the loads wait behind the operand traffic)
            auto load_slice = [&](int kt) {
                const uint32_t* s = p.sa + (long long)kt * p.R;
                return make_uint4(__ldg(s + rows[0]), __ldg(s + rows[1]), __ldg(s + rows[2]), __ldg(s + rows[3]));
            };
            uint4 q[MX_SCALE_AHEAD];
#pragma unroll
            for (int i = 0; i < MX_SCALE_AHEAD; ++i) q[i] = load_slice(min(i, p.k_tiles - 1));
            for (int kt0 = 0; ok && kt0 < p.k_tiles; kt0 += MX_SCALE_AHEAD) {
#pragma unroll
                for (int i = 0; i < MX_SCALE_AHEAD; ++i) {
                    const int kt = kt0 + i;
                    if (kt >= p.k_tiles) break;
                    const uint4 cur = q[i];
                    if (kt + MX_SCALE_AHEAD < p.k_tiles) q[i] = load_slice(kt + MX_SCALE_AHEAD);
                    if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag))) { ok = false; break; }
                    *reinterpret_cast<uint4*>(tiles_ptr + stage * MX_STAGE_BYTES + MX_A_BYTES + MX_B_BYTES + lane * 16) = cur;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->full[stage]));
                    if (++stage == MX_STAGES) { stage = 0; phase ^= 1u; }
                }
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
            if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag))) break;
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

// ---- the CTA-pair form ----------------------------------------------------------------------------------
// Two CTAs of a cluster share one 256-row x 208-column tile (tcgen05.mma.cta_group::2, M = 256): each keeps its own 128
// rows of A and 104 of the tile's weight rows in shared memory, so a K slice of 128 costs each SM 29 KB of operand
// loads against 58 KB per two 128 x 128 tiles of the single-CTA form, which the L2 -> SM path bounds.  208 columns, not
// 256: the two accumulators (tensor-memory columns 0 and 256) leave 48 columns behind each for three 16-column scale
// slots, one slot per ring stage.  A tile at the right edge is narrower (a multiple of 16 columns; the MMA's N is set
// per tile).
//   scale factors: each CTA holds the scales of its own 128 rows of A (4 columns) and of ALL the tile's weight rows (two
//   128-row blocks, 8 columns) in its own tensor memory; tcgen05.cp.cta_group::2, issued once, copies in both CTAs from
//   the same shared-memory offsets.  The weight-scale blocks of a (tile, K slice) are 1024 contiguous bytes in global
//   memory (a second copy of the scales in this tiling, written by the weight quantiser) and arrive by one tensor copy.
//   warp 0      TMA producer (both CTAs; all loads complete on the first CTA's full[stage], as in the bf16 pair kernels)
//   warp 1      first CTA: issues the MMAs and the commits for the pair
//   warp 2      activation scales of this CTA's 128 rows
//   warps 3..10 epilogue: 32-row slab x every other 32-column block (a 16-column remainder: plain stores)
//   warp 11     first CTA: issues the scale copies (smem -> tensor memory) of each stage
// What bounds it (cycle counters, throw-away builds): every tcgen05 instruction costs its issuing thread 60-85 cycles
// whatever its size, so a K slice (wait, four MMAs, commit) takes the MMA warp ~470 cycles -- more than the ~420 the
// tensor pipe needs for four N = 208 MMAs.  With the three scale copies in the same thread it was ~770; with two or four
// scale slots the chain MMA -> stage released -> copies -> MMA set the pace instead (~510).  In the full kernel a slice
// takes ~590 cycles: operand reads by the tensor core and fills by the TMA unit together ask shared memory for ~140 bytes
// per cycle at this tile width (halving the waits and commits per slice changed nothing).
constexpr int MXP_NT = 208;                 // tile columns over the pair
constexpr int MXP_ROWS = 2 * MX_BM;         // tile rows over the pair
constexpr int MXP_STAGES = 6;
constexpr int MXP_A_BYTES = MX_BM * MX_BK;              // 16 KB
constexpr int MXP_B_BYTES = (MXP_NT / 2) * MX_BK;       // 13 KB
constexpr int MXP_SFA_OFF = MXP_A_BYTES + MXP_B_BYTES;  // 512 bytes: this CTA's activation scales
constexpr int MXP_SFB_OFF = MXP_SFA_OFF + 512;          // 1024 bytes: the tile's weight scales
constexpr int MXP_STAGE_BYTES = 31 * 1024;              // 30.5 KB used; stages stay 1024-byte aligned
constexpr int MXP_TX_BYTES = MXP_A_BYTES + MXP_B_BYTES + 1024;   // bytes one CTA's loads deliver per stage
constexpr int MXP_EPI_WARPS = 8;
constexpr int MXP_COPY_WARP = 3 + MXP_EPI_WARPS;   // the scale-copy warp comes after the epilogue warps
constexpr int MXP_THREADS = 32 * (4 + MXP_EPI_WARPS);
constexpr int MXP_STAGING_BYTES = MXP_EPI_WARPS * 2048;
constexpr int MXP_ACC_STRIDE = 256;         // tensor-memory columns between the two accumulators
// one scale slot (16 columns) per ring stage, three behind each accumulator: a stage's slot is free when the stage is
__device__ __forceinline__ uint32_t mxp_slot_col(uint32_t stage) { return MXP_NT + (stage / 3u) * MXP_ACC_STRIDE + (stage % 3u) * 16; }
static_assert(MXP_STAGES == 6 && MXP_NT + 3 * 16 <= MXP_ACC_STRIDE, "scale slots");
static_assert(MXP_SFB_OFF + 1024 <= MXP_STAGE_BYTES, "stage layout");

struct MxPairCtl {
    unsigned long long full[MXP_STAGES];
    unsigned long long sf_full[MXP_STAGES];   // first CTA: the stage's scales are in tensor memory (and its operands landed)
    unsigned long long empty[MXP_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    unsigned long long drain_copy;
    uint32_t tmem_base;
    int abort_flag;
    int stage_n[MXP_STAGES];   // columns of the tile a stage belongs to (published by the first CTA's producer)
    int32_t offs[MX_MAX_E + 1];          // row-ragged form: offsets; weight gradients: slice_prefix
    int32_t tile_prefix[MX_MAX_E + 1];   // row-ragged form: 256-row tiles of the experts before e
};
constexpr int MXP_SMEM_BYTES = MXP_STAGES * MXP_STAGE_BYTES + MXP_STAGING_BYTES + 1024 + (int)sizeof(MxPairCtl);
static_assert(MXP_SMEM_BYTES <= 232448, "exceeds the shared memory a CTA can opt in to");

// The pair kernel serves two problems (template parameter WGRAD):
//   row-ragged GEMM   out[r, :] = a[r, :] . b[e]^T for the rows r of expert e: tiles of 256 rows from `offsets`, the
//                     contraction is k_tiles slices for every tile, b and its scale blocks are indexed by expert;
//   weight gradient   dW[e] [M, N] = A_e^T B_e with token-quantised, transposed operands (further down): a fixed tile
//                     list (expert x M tiles x N tiles), the contraction of expert e is the slices
//                     [slice_prefix[e], slice_prefix[e + 1]) of both operands, nothing is indexed by expert but the output.
struct MxPairParams {
    const int32_t* prefix;   // offsets [E + 1] / slice_prefix [E + 1]
    int E, k_tiles, n_tiles, m_tiles, n_cols, n_slices;   // k_tiles: row-ragged form; m_tiles, n_slices: weight gradients
    int M;                   // weight gradients: rows of one expert's output
    long long sa_rows;       // rows per slice of the A-side scale words: R / M
    const uint32_t* sa;      // scale words of the A side [slices][sa_rows]
    bf16* out;
    long long ldo;
};

__device__ __forceinline__ uint32_t mxp_idesc(uint32_t n, uint32_t sf) {
    return (sf << 4) | ((n >> 3) << 17) | (1u << 23) | ((uint32_t)(MXP_ROWS >> 4) << 24) | (sf << 29);
}
__device__ __forceinline__ void mxp_copy_scales(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void mxp_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa,
                                        uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.u32 p, %4, 0;"
        " tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p; }" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
}
// one lane of the (converged) warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred = 0;
    asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; @p mov.u32 %0, 1; }" : "+r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t v[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

struct MxPairTile {
    int e, row0, row_end;   // first row of the tile and end of the valid rows, as the A operand counts them
    int out_shift;          // output row = A row + out_shift
    int n0, nt, width;      // first column, column-tile index, columns
    int k0, k_tiles;        // K slices [k0, k0 + k_tiles) of both operands
    int b_row, sfb_row0;    // first row of the tile in the B codes; row of its first scale block
};
template <bool WGRAD>
__device__ __forceinline__ MxPairTile mxp_decode(const MxPairParams& p, const MxPairCtl* ctl, long long t) {
    MxPairTile tl;
    if (WGRAD) {
        const int per_e = p.m_tiles * p.n_tiles;
        tl.e = (int)(t / per_e);
        const int local = (int)(t - (long long)tl.e * per_e);
        tl.nt = local / p.m_tiles;   // column tile major inside an expert: the pairs running together share the B tile in L2
        tl.row0 = (local - tl.nt * p.m_tiles) * MXP_ROWS;
        tl.row_end = p.M;
        tl.out_shift = tl.e * p.M;
        tl.k0 = ctl->offs[tl.e];
        tl.k_tiles = ctl->offs[tl.e + 1] - tl.k0;
        tl.n0 = tl.nt * MXP_NT;
        tl.b_row = tl.n0;
        tl.sfb_row0 = tl.nt * p.n_slices + tl.k0;
    } else {
        int lo = 0, hi = p.E;   // largest e with tile_prefix[e] * n_tiles <= t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((long long)ctl->tile_prefix[mid] * p.n_tiles <= t) lo = mid; else hi = mid;
        }
        const int local = (int)(t - (long long)ctl->tile_prefix[lo] * p.n_tiles);
        const int m_tiles_e = ctl->tile_prefix[lo + 1] - ctl->tile_prefix[lo];
        tl.e = lo;
        tl.nt = local / m_tiles_e;   // column tile major inside an expert (the pairs running together share weight tiles in L2)
        tl.row0 = ctl->offs[lo] + (local - tl.nt * m_tiles_e) * MXP_ROWS;
        tl.row_end = ctl->offs[lo + 1];
        tl.out_shift = 0;
        tl.k0 = 0;
        tl.k_tiles = p.k_tiles;
        tl.n0 = tl.nt * MXP_NT;
        tl.b_row = lo * p.n_cols + tl.n0;
        tl.sfb_row0 = (lo * p.n_tiles + tl.nt) * p.k_tiles;
    }
    tl.width = min(MXP_NT, p.n_cols - tl.n0);
    return tl;
}
// K slices of tile t (the roles that do not need the rest of the tile)
template <bool WGRAD>
__device__ __forceinline__ int mxp_k_tiles(const MxPairParams& p, const MxPairCtl* ctl, long long t) {
    if (!WGRAD) return p.k_tiles;
    const int e = (int)(t / ((long long)p.m_tiles * p.n_tiles));
    return ctl->offs[e + 1] - ctl->offs[e];
}

template <bool WGRAD>
__global__ void __launch_bounds__(MXP_THREADS, 1)
mx_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_sfb, const __grid_constant__ CUtensorMap map_o,
                    const MxPairParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
    MxPairCtl* ctl = reinterpret_cast<MxPairCtl*>(tiles_ptr + MXP_STAGES * MXP_STAGE_BYTES + MXP_STAGING_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();   // 0 = the CTA that issues the MMAs
    const long long first_tile = blockIdx.x >> 1, tile_stride = gridDim.x >> 1;

    for (int e = threadIdx.x; e <= p.E; e += MXP_THREADS) ctl->offs[e] = p.prefix[e];
    if (threadIdx.x == 0) {
        for (int s = 0; s < MXP_STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 4);   // per CTA: the producer's arrive (with its byte count) + the scale warp's
            mbar_init(smem_u32(&ctl->sf_full[s]), 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctl->tmem_full[a]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[a]), 2 * MXP_EPI_WARPS);
        }
        mbar_init(smem_u32(&ctl->drain), 1);
        mbar_init(smem_u32(&ctl->drain_copy), 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
        prefetch_tmap(&map_sfb);
        prefetch_tmap(&map_o);
    }
    __syncthreads();
    if (!WGRAD && threadIdx.x == 0) {   // row-ragged form: tiles of 256 rows per expert
        int run = 0;
        for (int e = 0; e < p.E; ++e) {
            ctl->tile_prefix[e] = run;
            run += (ctl->offs[e + 1] - ctl->offs[e] + MXP_ROWS - 1) / MXP_ROWS;
        }
        ctl->tile_prefix[p.E] = run;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"((uint32_t)MX_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the other CTA's barriers and tensor memory exist from here on
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const long long n_tiles_total = WGRAD ? (long long)p.E * p.m_tiles * p.n_tiles : (long long)ctl->tile_prefix[p.E] * p.n_tiles;
    const uint32_t full0 = map_to_cta(smem_u32(&ctl->full[0]), 0);   // full[] of the MMA-issuing CTA

    if (warp == 0) {
        // ================= producer (both CTAs; each fills its own ring) =================
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (long long t = first_tile; ok && t < n_tiles_total; t += tile_stride) {
                const MxPairTile tl = mxp_decode<WGRAD>(p, ctl, t);
                const int sfb_row0 = tl.sfb_row0;
                const int b_row = tl.b_row + (int)rank * (tl.width >> 1);
                for (int kt = 0; kt < tl.k_tiles; ++kt) {
                    if (!mx_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
#ifdef MOE_TEST_HOOKS
                    if (g_mx_test_withhold_first_stage != 0 && issued == 0) {
                        ++issued;
                        if (++stage == MXP_STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
#endif
                    if (rank == 0) ctl->stage_n[stage] = tl.width;   // read by the MMA thread after its wait on full[stage]
                    const uint32_t bar = full0 + stage * (uint32_t)sizeof(unsigned long long);
                    const uint32_t dst = tiles_base + stage * MXP_STAGE_BYTES;
                    mbar_arrive_expect_tx_cluster(bar, MXP_TX_BYTES);
                    tma_load_2d_pair(dst, &map_a, (tl.k0 + kt) * MX_BK, tl.row0 + (int)rank * MX_BM, bar);
                    tma_load_2d_pair(dst + MXP_A_BYTES, &map_b, (tl.k0 + kt) * MX_BK, b_row, bar);
                    tma_load_2d_pair(dst + MXP_SFB_OFF, &map_sfb, 0, sfb_row0 + kt, bar);
                    ++issued;
                    if (++stage == MXP_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok && issued != 0) {
                // leave no bulk copy in flight: the copies report to a barrier this thread cannot always poll (the other
                // CTA's), so outwait them -- a copy that was issued completes within microseconds
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer: the first CTA's warp 1 =================
        // The whole warp runs the loop and takes every wait's verdict together; one elected lane issues the tcgen05
        // instructions.  (Measured against the same loop under `if (lane == 0)`: no difference in time -- the 60-85
        // cycles a tcgen05 instruction costs its issuer are not operand marshalling.)
        if (rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0, n = MXP_NT;
            bool ok = true;
            for (long long t = first_tile; ok && t < n_tiles_total; t += tile_stride) {
                const int k_tiles_t = mxp_k_tiles<WGRAD>(p, ctl, t);
                if (k_tiles_t == 0) continue;   // (weight gradients) an expert without rows: the epilogue writes zeros on its own
                if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * MXP_ACC_STRIDE;
                for (int kt = 0; kt < k_tiles_t; ++kt) {
                    if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->sf_full[stage]), phase, abort_flag))) { ok = false; break; }
                    tc_fence_after();
                    if (kt == 0) n = (uint32_t)ctl->stage_n[stage];
                    const uint32_t s_base = tiles_base + stage * MXP_STAGE_BYTES;
                    const uint32_t sfa_t = tmem_base + mxp_slot_col(stage), sfb_t = sfa_t + 4;
                    const uint64_t a_desc = mx_operand_desc(s_base), b_desc = mx_operand_desc(s_base + MXP_A_BYTES);
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < MX_BK / 32; ++k)
                            mxp_mma(d_tmem, a_desc + (uint64_t)((k * 32) >> 4), b_desc + (uint64_t)((k * 32) >> 4), mxp_idesc(n, k),
                                    sfa_t, sfb_t, (kt != 0 || k != 0) ? 1u : 0u);
                        tc_commit<true>(smem_u32(&ctl->empty[stage]));
                    }
                    __syncwarp();
                    if (++stage == MXP_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit<true>(smem_u32(&ctl->tmem_full[acc]));
                __syncwarp();
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            // all issued MMAs must have retired before tensor memory is released
            if (lane == 0) {
                tc_commit_local<true>(smem_u32(&ctl->drain));
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < WAIT_LIMIT_NS) {}
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ================= activation scales of this CTA's 128 rows =================
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (long long t = first_tile; ok && t < n_tiles_total; t += tile_stride) {
            const MxPairTile tl = mxp_decode<WGRAD>(p, ctl, t);
            long long rows[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const long long r = (long long)tl.row0 + (int)rank * MX_BM + 32 * i + lane;
                rows[i] = r < p.sa_rows ? r : p.sa_rows - 1;   // rows past the end are never stored; any valid address will do
            }
            // the words of MX_SCALE_AHEAD slices are in flight at any time: one slice per global-load round trip would
            // bound the whole pipeline (the loads wait behind the operand traffic)
            auto load_slice = [&](int kt) {
                const uint32_t* s = p.sa + (long long)(tl.k0 + kt) * p.sa_rows;
                return make_uint4(__ldg(s + rows[0]), __ldg(s + rows[1]), __ldg(s + rows[2]), __ldg(s + rows[3]));
            };
            uint4 q[MX_SCALE_AHEAD];
#pragma unroll
            for (int i = 0; i < MX_SCALE_AHEAD; ++i) q[i] = load_slice(min(i, max(tl.k_tiles - 1, 0)));
            for (int kt0 = 0; ok && kt0 < tl.k_tiles; kt0 += MX_SCALE_AHEAD) {
#pragma unroll
                for (int i = 0; i < MX_SCALE_AHEAD; ++i) {
                    const int kt = kt0 + i;
                    if (kt >= tl.k_tiles) break;
                    const uint4 cur = q[i];
                    if (kt + MX_SCALE_AHEAD < tl.k_tiles) q[i] = load_slice(kt + MX_SCALE_AHEAD);
                    if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag))) { ok = false; break; }
                    *reinterpret_cast<uint4*>(tiles_ptr + stage * MXP_STAGE_BYTES + MXP_SFA_OFF + lane * 16) = cur;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(full0 + stage * (uint32_t)sizeof(unsigned long long));
                    if (++stage == MXP_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == MXP_COPY_WARP) {
        // ================= scale copies: one thread of the first CTA =================
        // Takes the three tcgen05.cp per K slice off the MMA thread (each tcgen05 instruction costs the issuing thread
        // 60-85 cycles; with them the MMA thread needed ~770 cycles per slice).  Every ring stage has its own scale slot in
        // tensor memory: full[stage] can only complete after the stage was released, i.e. after the MMAs that read the
        // slot's previous contents have completed.
        if (rank == 0 && lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long t = first_tile; ok && t < n_tiles_total; t += tile_stride) {
                const int k_tiles_t = mxp_k_tiles<WGRAD>(p, ctl, t);
                for (int kt = 0; kt < k_tiles_t; ++kt) {
                    if (!mx_wait(smem_u32(&ctl->full[stage]), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t s_base = tiles_base + stage * MXP_STAGE_BYTES;
                    const uint32_t sfa_t = tmem_base + mxp_slot_col(stage), sfb_t = sfa_t + 4;
                    mxp_copy_scales(sfa_t, mx_scale_desc(s_base + MXP_SFA_OFF));
                    mxp_copy_scales(sfb_t, mx_scale_desc(s_base + MXP_SFB_OFF));
                    mxp_copy_scales(sfb_t + 4, mx_scale_desc(s_base + MXP_SFB_OFF + 512));
                    tc_commit_local<true>(smem_u32(&ctl->sf_full[stage]));
                    if (++stage == MXP_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // all issued copies must have retired before tensor memory is released
            tc_commit_local<true>(smem_u32(&ctl->drain_copy));
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&ctl->drain_copy), 0) && global_timer_ns() - t0 < WAIT_LIMIT_NS) {}
        }
        __syncwarp();
    } else {
        // ================= epilogue (warps 3..10, both CTAs) =================
        const int quarter = warp & 3;          // tensor-memory lanes [32 * quarter, 32 * quarter + 32)
        const int half = (warp - 3) >> 2;      // 32-column blocks 0, 2, 4, 6 or 1, 3, 5 (+ the 16-column tail)
        uint8_t* stage_ptr = tiles_ptr + MXP_STAGES * MXP_STAGE_BYTES + (warp - 3) * 2048;
        const int sw = (lane >> 1) & 3;
        const uint32_t empty0 = map_to_cta(smem_u32(&ctl->tmem_empty[0]), 0);
        uint32_t n_stores = 0, acc = 0, acc_phase = 0;
        for (long long t = first_tile; t < n_tiles_total; t += tile_stride) {
            const MxPairTile tl = mxp_decode<WGRAD>(p, ctl, t);
            const bool have_acc = tl.k_tiles != 0;
            if (have_acc) {
                if (!__all_sync(0xffffffffu, mx_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag))) break;
                tc_fence_after();
            }
            const uint32_t taddr = tmem_base + acc * MXP_ACC_STRIDE + ((uint32_t)(quarter * 32) << 16);
            const int slab_in = tl.row0 + (int)rank * MX_BM + quarter * 32;   // first row of this warp's slab, as the A operand counts rows
            const int rows_valid = max(0, min(32, tl.row_end - slab_in));
            const int slab0 = slab_in + tl.out_shift;                         // ... and as the output does
#pragma unroll 1
            for (int c = half; c < 8; c += 2) {
                const int left = tl.width - 32 * c;   // columns of the tile from this block on (warp-uniform)
                if (left <= 0) break;
                const int n = tl.n0 + c * 32;
                uint32_t w[16];
                if (!have_acc) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) w[j] = 0u;
                } else if (left >= 32) {
                    uint32_t v[32];
                    tc_ld32(taddr + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) w[j] = pack_bf16(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                } else {
                    uint32_t v[16];
                    tc_ld16(taddr + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 8; ++j) w[j] = pack_bf16(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                }
                if (rows_valid == 0) continue;
                if (left >= 32 && rows_valid == 32) {
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
                    d4[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    d4[1] = make_uint4(w[4], w[5], w[6], w[7]);
                    if (left >= 32) {
                        d4[2] = make_uint4(w[8], w[9], w[10], w[11]);
                        d4[3] = make_uint4(w[12], w[13], w[14], w[15]);
                    }
                }
            }
            if (!have_acc) continue;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(empty0 + acc * (uint32_t)sizeof(unsigned long long));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (n_stores != 0 && lane == 0) bulk_wait_all0();
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // neither CTA's shared memory / barriers may go away while the other still uses them
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)MX_TMEM_COLS) : "memory");
    }
}

// ---- quantisers ---------------------------------------------------------------------------------------
// scale exponent of a block with largest magnitude amax: floor(log2 amax) - 8, clamped to the E8M0 range; -127 for zero
__device__ __forceinline__ int mx_scale_exp(float amax) {
    if (!(amax > 0.f)) return -127;
    const int field = (__float_as_int(amax) >> 23) & 0xFF;             // amax is positive and finite
    const int e = (field != 0 ? field - 127 : ilogbf(amax)) - 8;       // subnormal magnitudes take the library route
    return e < -127 ? -127 : (e > 127 ? 127 : e);
}
// 2^-s as a float (s in [-127, 127]; 2^-127 is a subnormal)
__device__ __forceinline__ float mx_inv_scale(int s) {
    return s == 127 ? __int_as_float(0x00400000) : __int_as_float((127 - s) << 23);
}
// two values -> two codes (the first in the low byte), one conversion instruction
__device__ __forceinline__ uint32_t mx_e4m3x2(float lo, float hi) {
    return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);
}

// rows x n bf16 -> codes (same layout) and scales.  A warp takes two (row, 128-wide slice) units per load: lane l holds
// the 8 elements 8l..8l+7 of the 256 contiguous ones (one 16-byte load), the 4 lanes of a block of 32 agree on its scale
// through two shuffles; four such loads are in flight per lane.  The 4 scale bytes of a (row, slice) are one 32-bit word:
//   WEIGHTS = false (activations): word [slice][row];
//   WEIGHTS = true  (weights whose contraction axis is contiguous, rows = E * n_feat, e.g. W_down read as [I, H] for the
//                    data gradient): the word's place in each of the two weight-scale tilings.  The output may be a
//                    column range of a wider operand (out_k_tiles slices per row, this input filling slices
//                    out_kt0 .. out_kt0 + n/128): W_gate and W_up side by side along the contraction of the gate/up
//                    data gradient.
template <bool WEIGHTS>
__global__ void __launch_bounds__(256) mx_quantize_rows_kernel(const uint4* __restrict__ x, long long rows, int n, int n_feat,
                                                               int out_k_tiles, int out_kt0, uint2* __restrict__ codes,
                                                               uint8_t* __restrict__ scales, uint8_t* __restrict__ scales_pair) {
    constexpr int U = 4;
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const int k_tiles = n / 128;
    const long long total = rows * k_tiles;            // units of 128 elements, contiguous in memory
    const long long pairs = (total + 1) / 2;
    const int n_tiles_p = WEIGHTS ? (n_feat + MXP_NT - 1) / MXP_NT : 0;
    for (long long p0 = warp * U; p0 < pairs; p0 += n_warps * U) {
        uint4 raw[U];
#pragma unroll
        for (int i = 0; i < U; ++i) {
            const long long u = 2 * (p0 + i) + (lane >> 4);
            raw[i] = (u < total) ? __ldg(x + (p0 + i) * 32 + lane) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < U; ++i) {
            if (p0 + i >= pairs) break;
            const long long u = 2 * (p0 + i) + (lane >> 4);   // this half-warp's unit
            const uint32_t* rw = reinterpret_cast<const uint32_t*>(&raw[i]);
            float v[8];
            float amax = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&rw[j]));
                v[2 * j] = f.x; v[2 * j + 1] = f.y;
                amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            const int se = mx_scale_exp(amax);
            const float inv = mx_inv_scale(se);
            uint2 out;
            out.x = mx_e4m3x2(v[0] * inv, v[1] * inv) | (mx_e4m3x2(v[2] * inv, v[3] * inv) << 16);
            out.y = mx_e4m3x2(v[4] * inv, v[5] * inv) | (mx_e4m3x2(v[6] * inv, v[7] * inv) << 16);
            const long long r = (total >> 32) == 0 ? (long long)((uint32_t)u / (uint32_t)k_tiles) : u / k_tiles;
            const int kt = (int)(u - r * k_tiles) + out_kt0;
            if (u < total) codes[(r * out_k_tiles + kt) * 16 + (lane & 15)] = out;
            const uint32_t sbyte = (uint32_t)(se + 127);
            const int base = lane & 16;                       // first lane of this half-warp
            const uint32_t word = __shfl_sync(0xffffffffu, sbyte, base) | (__shfl_sync(0xffffffffu, sbyte, base + 4) << 8) |
                                  (__shfl_sync(0xffffffffu, sbyte, base + 8) << 16) | (__shfl_sync(0xffffffffu, sbyte, base + 12) << 24);
            if ((lane & 15) == 0 && u < total) {
                if (!WEIGHTS) {
                    reinterpret_cast<uint32_t*>(scales)[(long long)kt * rows + r] = word;
                } else {
                    const int e = (int)(r / n_feat), f = (int)(r - (long long)e * n_feat);
                    *reinterpret_cast<uint32_t*>(scales + (((long long)e * (n_feat / 128) + f / 128) * out_k_tiles + kt) * 512 +
                                                 (f % 32) * 16 + ((f % 128) / 32) * 4) = word;
                    const int nt = f / MXP_NT, c = f % MXP_NT;
                    *reinterpret_cast<uint32_t*>(scales_pair + (((long long)e * n_tiles_p + nt) * out_k_tiles + kt) * 1024 +
                                                 (c >> 7) * 512 + (c % 32) * 16 + ((c % 128) / 32) * 4) = word;
                }
            }
        }
    }
}

// The SwiGLU activation of saved pre-activations with the activation quantiser fused in: GU [rows, 2I] bf16 ->
// H_act [rows, I] bf16 (silu(g) * u in fp32, rounded once) and the block-scaled FP8 codes and scale words of exactly those
// bf16 values, in the layouts of the activation quantiser.  Same lane mapping as mx_quantize_rows_kernel: a half-warp per
// (row, 128-wide slice of I), 8 elements per lane.
__global__ void __launch_bounds__(256) mx_swiglu_quantize_kernel(const uint4* __restrict__ gu, long long rows, int I,
                                                                 uint4* __restrict__ h_act, uint2* __restrict__ codes,
                                                                 uint32_t* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const int k_tiles = I / 128;
    const long long total = rows * k_tiles;
    const long long pairs = (total + 1) / 2;
    for (long long p0 = warp; p0 < pairs; p0 += n_warps) {
        const long long u = 2 * p0 + (lane >> 4);
        if (u >= total) continue;   // only the last pair can be half empty; no warp-wide operation below needs those lanes
        const long long r = (total >> 32) == 0 ? (long long)((uint32_t)u / (uint32_t)k_tiles) : u / k_tiles;
        const int kt = (int)(u - r * k_tiles);
        const long long g_idx = (r * 2 * I + kt * 128) / 8 + (lane & 15);
        const uint4 graw = __ldg(gu + g_idx), uraw = __ldg(gu + g_idx + I / 8);
        const uint32_t* gw = reinterpret_cast<const uint32_t*>(&graw);
        const uint32_t* uw = reinterpret_cast<const uint32_t*>(&uraw);
        uint32_t hw[4];
        float v[8];
        float amax = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 g2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[j]));
            const float2 u2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&uw[j]));
            const float h0 = __fdividef(g2.x, 1.f + __expf(-g2.x)) * u2.x;
            const float h1 = __fdividef(g2.y, 1.f + __expf(-g2.y)) * u2.y;
            hw[j] = pack_bf16(h0, h1);
            const float2 hr = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hw[j]));   // what H_act holds
            v[2 * j] = hr.x; v[2 * j + 1] = hr.y;
            amax = fmaxf(amax, fmaxf(fabsf(hr.x), fabsf(hr.y)));
        }
        const uint32_t half_mask = (lane & 16) ? 0xffff0000u : 0x0000ffffu;
        amax = fmaxf(amax, __shfl_xor_sync(half_mask, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(half_mask, amax, 2));
        const int se = mx_scale_exp(amax);
        const float inv = mx_inv_scale(se);
        uint2 out;
        out.x = mx_e4m3x2(v[0] * inv, v[1] * inv) | (mx_e4m3x2(v[2] * inv, v[3] * inv) << 16);
        out.y = mx_e4m3x2(v[4] * inv, v[5] * inv) | (mx_e4m3x2(v[6] * inv, v[7] * inv) << 16);
        h_act[u * 16 + (lane & 15)] = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        codes[u * 16 + (lane & 15)] = out;
        const uint32_t sbyte = (uint32_t)(se + 127);
        const int base = lane & 16;
        const uint32_t word = __shfl_sync(half_mask, sbyte, base) | (__shfl_sync(half_mask, sbyte, base + 4) << 8) |
                              (__shfl_sync(half_mask, sbyte, base + 8) << 16) | (__shfl_sync(half_mask, sbyte, base + 12) << 24);
        if ((lane & 15) == 0) scales[(long long)kt * rows + r] = word;
    }
}

// The SwiGLU backward (elementwise part of the gate/up backward) with the row quantiser of its result fused in:
// dGU = [dg | du] [rows, 2I] bf16 exactly as moe_swiglu_bwd computes it, and the block-scaled FP8 codes and scale words of
// those bf16 values along the 2I columns (the A operand of the FP8 gate/up dgrad).  One thread per 8 columns of a row
// (its 8 gate and its 8 up columns), a half-warp per 128-wide slice of each half.
__global__ void __launch_bounds__(256) mx_swiglu_bwd_quantize_kernel(const uint4* __restrict__ dh_act, const uint4* __restrict__ gu,
                                                                     long long rows, int I, uint4* __restrict__ dgu,
                                                                     uint2* __restrict__ codes, uint32_t* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int iv = I >> 3;                       // 16-byte pieces per half row (a multiple of 16)
    if (i >= rows * iv) return;                  // whole half-warps leave together
    const long long r = (rows * iv >> 32) == 0 ? (long long)((uint32_t)i / (uint32_t)iv) : i / iv;
    const int c = (int)(i - r * iv);
    const uint4 dhv = __ldg(dh_act + i), gv = __ldg(gu + r * (2 * iv) + c), uv = __ldg(gu + r * (2 * iv) + iv + c);
    const uint32_t* dw = reinterpret_cast<const uint32_t*>(&dhv);
    const uint32_t* gw = reinterpret_cast<const uint32_t*>(&gv);
    const uint32_t* uw = reinterpret_cast<const uint32_t*>(&uv);
    uint32_t og[4], ou[4];
    float vg[8], vu[8], amax_g = 0.f, amax_u = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 d2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&dw[j]));
        const float2 g2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[j]));
        const float2 u2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&uw[j]));
        const float s0 = __fdividef(1.f, 1.f + __expf(-g2.x)), s1 = __fdividef(1.f, 1.f + __expf(-g2.y));
        og[j] = pack_bf16(d2.x * u2.x * s0 * (1.f + g2.x * (1.f - s0)), d2.y * u2.y * s1 * (1.f + g2.y * (1.f - s1)));
        ou[j] = pack_bf16(d2.x * g2.x * s0, d2.y * g2.y * s1);
        const float2 rg = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&og[j]));   // what dGU holds
        const float2 ru = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ou[j]));
        vg[2 * j] = rg.x; vg[2 * j + 1] = rg.y; vu[2 * j] = ru.x; vu[2 * j + 1] = ru.y;
        amax_g = fmaxf(amax_g, fmaxf(fabsf(rg.x), fabsf(rg.y)));
        amax_u = fmaxf(amax_u, fmaxf(fabsf(ru.x), fabsf(ru.y)));
    }
    dgu[r * (2 * iv) + c] = make_uint4(og[0], og[1], og[2], og[3]);
    dgu[r * (2 * iv) + iv + c] = make_uint4(ou[0], ou[1], ou[2], ou[3]);
    const uint32_t half_mask = (lane & 16) ? 0xffff0000u : 0x0000ffffu;
    amax_g = fmaxf(amax_g, __shfl_xor_sync(half_mask, amax_g, 1));
    amax_g = fmaxf(amax_g, __shfl_xor_sync(half_mask, amax_g, 2));
    amax_u = fmaxf(amax_u, __shfl_xor_sync(half_mask, amax_u, 1));
    amax_u = fmaxf(amax_u, __shfl_xor_sync(half_mask, amax_u, 2));
    const int se_g = mx_scale_exp(amax_g), se_u = mx_scale_exp(amax_u);
    const float inv_g = mx_inv_scale(se_g), inv_u = mx_inv_scale(se_u);
    uint2 cg, cu;
    cg.x = mx_e4m3x2(vg[0] * inv_g, vg[1] * inv_g) | (mx_e4m3x2(vg[2] * inv_g, vg[3] * inv_g) << 16);
    cg.y = mx_e4m3x2(vg[4] * inv_g, vg[5] * inv_g) | (mx_e4m3x2(vg[6] * inv_g, vg[7] * inv_g) << 16);
    cu.x = mx_e4m3x2(vu[0] * inv_u, vu[1] * inv_u) | (mx_e4m3x2(vu[2] * inv_u, vu[3] * inv_u) << 16);
    cu.y = mx_e4m3x2(vu[4] * inv_u, vu[5] * inv_u) | (mx_e4m3x2(vu[6] * inv_u, vu[7] * inv_u) << 16);
    codes[r * (2 * iv) + c] = cg;
    codes[r * (2 * iv) + iv + c] = cu;
    const int base = lane & 16;
    const uint32_t bg = (uint32_t)(se_g + 127), bu = (uint32_t)(se_u + 127);
    const uint32_t word_g = __shfl_sync(half_mask, bg, base) | (__shfl_sync(half_mask, bg, base + 4) << 8) |
                            (__shfl_sync(half_mask, bg, base + 8) << 16) | (__shfl_sync(half_mask, bg, base + 12) << 24);
    const uint32_t word_u = __shfl_sync(half_mask, bu, base) | (__shfl_sync(half_mask, bu, base + 4) << 8) |
                            (__shfl_sync(half_mask, bu, base + 8) << 16) | (__shfl_sync(half_mask, bu, base + 12) << 24);
    if ((lane & 15) == 0) {
        const int kt = c >> 4;                   // 128-wide slice inside the half
        scales[(long long)kt * rows + r] = word_g;
        scales[(long long)((I >> 7) + kt) * rows + r] = word_u;
    }
}

// Weights whose OUTPUT-feature axis is contiguous: w [E, k, n] bf16 (W_down [E, I, H]; W_gate, W_up [E, H, I]) -> codes
// transposed, contraction contiguous, as rows n_off .. n_off + n of [E, n_total, k] (W_gate and W_up stacked along the 2I
// output features of the gate/up projection), and the scale bytes in both tilings.  One thread per (expert, block of
// 32 along k, feature): consecutive lanes take consecutive features, so the 32 loads of a thread are coalesced across
// the warp; the thread keeps the 32 values, picks the scale and writes 32 contiguous code bytes.
__global__ void __launch_bounds__(256) mx_quantize_w_transposed_kernel(const bf16* __restrict__ w, int E, int k, int n,
                                                                       int n_total, int n_off, uint8_t* __restrict__ codes,
                                                                       uint8_t* __restrict__ scales,
                                                                       uint8_t* __restrict__ scales_pair) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int blocks_k = k / 32;
    const long long total = (long long)E * blocks_k * n;
    if (idx >= total) return;
    const int h = (int)(idx % n);
    const int ib = (int)((idx / n) % blocks_k);
    const int e = (int)(idx / ((long long)n * blocks_k));
    const bf16* src = w + ((long long)e * k + (long long)ib * 32) * n + h;
    float v[32];
    float amax = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        v[j] = __bfloat162float(src[(long long)j * n]);
        amax = fmaxf(amax, fabsf(v[j]));
    }
    const int se = mx_scale_exp(amax);
    const float inv = mx_inv_scale(se);
    uint32_t out[8];
#pragma unroll
    for (int q = 0; q < 8; ++q)
        out[q] = mx_e4m3x2(v[4 * q] * inv, v[4 * q + 1] * inv) | (mx_e4m3x2(v[4 * q + 2] * inv, v[4 * q + 3] * inv) << 16);
    const int f = n_off + h;   // output feature of the GEMM
    uint4* dst = reinterpret_cast<uint4*>(codes + ((long long)e * n_total + f) * k + (long long)ib * 32);
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
    const int k_tiles = k / 128;
    scales[(((long long)e * (n_total / 128) + f / 128) * k_tiles + ib / 4) * 512 + (f % 32) * 16 + ((f % 128) / 32) * 4 + (ib % 4)] =
        (uint8_t)(se + 127);
    // the same byte in the tiling of the CTA-pair kernel: per (208-column tile, K slice) two 512-byte blocks
    const int nt = f / MXP_NT, c = f % MXP_NT;
    const int n_tiles_p = (n_total + MXP_NT - 1) / MXP_NT;
    scales_pair[(((long long)e * n_tiles_p + nt) * k_tiles + ib / 4) * 1024 + (c >> 7) * 512 + (c % 32) * 16 + ((c % 128) / 32) * 4 +
                (ib % 4)] = (uint8_t)(se + 127);
}


// ---- token-axis quantiser (operands of the weight gradients) ---------------------------------------------
// dW[e] [M, N] = Q(A_e)^T Q(B_e) over the rows of expert e, both operands quantised along the token axis in blocks of 32
// rows counted from the expert's first row and stored TRANSPOSED, contraction contiguous: codes [features, pitch] where
// column slice_prefix[e] * 128 + i holds row offsets[e] + i of the packed tensor and every expert's columns are padded
// with zero codes to a multiple of 128 -- so a K slice of 128 columns belongs to exactly one expert, both operands are
// K-major like everywhere else in this file, and the ragged contraction needs no clearing of foreign rows in shared
// memory.  The tile list is fixed (every expert x M tiles x N tiles); an expert's K slices are
// [slice_prefix[e], slice_prefix[e+1]); a tile of an expert without rows skips the pipeline and its epilogue writes zeros.
// slice_prefix[e] = number of 128-row slices of the experts before e, every expert's rows rounded up to whole slices
__global__ void __launch_bounds__(1024) mx_slice_prefix_kernel(const int32_t* __restrict__ offsets, int E, int32_t* __restrict__ sp) {
    __shared__ int32_t part[32];
    const int e = threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int v = (e < E) ? (offsets[e + 1] - offsets[e] + 127) >> 7 : 0;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) part[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = part[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += t;
        }
        part[lane] = w;
    }
    __syncthreads();
    const int before = incl - v + (warp > 0 ? part[warp - 1] : 0);
    if (e < E) sp[e] = before;
    if (e == E - 1) sp[E] = before + v;
}

// x [R, ld] bf16, columns [col0, col0 + n) -> codes_t [n, pitch] (transposed, zero-padded per expert), scale words
// [pitch/128][n] (the operand as the M side) and scale blocks in the pair tiling [ceil(n/208)][pitch/128][1024] (the
// operand as the N side).  One thread per (128-column slice, group of 8 features): the slice's four blocks of 32 rows one
// after the other -- a 16-byte load per row, 512 contiguous bytes per warp; the thread keeps the 32 x 8 values as
// loaded, finds the 8 block maxima, writes 32 code bytes per feature -- then the four scale bytes of each feature as
// one word into each of the two scale layouts.
__global__ void __launch_bounds__(128) mx_quantize_tokens_kernel(const bf16* __restrict__ x, long long ld, int col0, int n,
                                                                 const int32_t* __restrict__ offsets, const int32_t* __restrict__ sp,
                                                                 int E, long long pitch, uint8_t* __restrict__ codes_t,
                                                                 uint8_t* __restrict__ sa_words, uint8_t* __restrict__ sb_atoms) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int groups = n >> 3;
    const int f0 = (int)(idx % groups) * 8;
    const int slice = (int)(idx / groups);
    if (slice >= sp[E]) return;
    int lo = 0, hi = E;                                 // the expert whose slices hold `slice`: largest e with sp[e] <= slice
    while (hi - lo > 1) {                               // (experts without rows share their successor's prefix)
        const int mid = (lo + hi) >> 1;
        if (sp[mid] <= slice) lo = mid; else hi = mid;
    }
    const int e = lo;
    const int n_e = offsets[e + 1] - offsets[e];
    const long long ld16 = ld >> 3;
    uint32_t words[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) words[q] = 0u;
#pragma unroll 1
    for (int blk = 0; blk < 4; ++blk) {
        const int local_block = 4 * (slice - sp[e]) + blk;
        const long long pb = 4ll * slice + blk;         // padded block of 32 rows
        const int valid = max(0, min(32, n_e - 32 * local_block));
        const uint4* src = reinterpret_cast<const uint4*>(x + ((long long)offsets[e] + 32ll * local_block) * ld + col0 + f0);
        uint4 raw[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) raw[j] = j < valid ? __ldg(src + (long long)j * ld16) : make_uint4(0u, 0u, 0u, 0u);
        float amax[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) amax[q] = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw[j]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[q]));
                amax[2 * q] = fmaxf(amax[2 * q], fabsf(v.x));
                amax[2 * q + 1] = fmaxf(amax[2 * q + 1], fabsf(v.y));
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int se = mx_scale_exp(amax[q]);
            const float inv = mx_inv_scale(se);
            uint32_t out[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) {      // rows 4g .. 4g+3 of feature f0 + q
                float v[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t w = reinterpret_cast<const uint32_t*>(&raw[4 * g + t])[q >> 1];
                    v[t] = __uint_as_float((q & 1) ? (w & 0xffff0000u) : (w << 16));      // bf16 -> fp32 is a shift
                }
                out[g] = mx_e4m3x2(v[0] * inv, v[1] * inv) | (mx_e4m3x2(v[2] * inv, v[3] * inv) << 16);
            }
            uint4* dst = reinterpret_cast<uint4*>(codes_t + (long long)(f0 + q) * pitch + pb * 32);
            dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
            dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
            words[q] |= (uint32_t)(se + 127) << (8 * blk);
        }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int f = f0 + q;
        *reinterpret_cast<uint32_t*>(sa_words + ((long long)slice * n + f) * 4) = words[q];
        const int nt = f / MXP_NT, c = f % MXP_NT;
        *reinterpret_cast<uint32_t*>(sb_atoms + ((long long)nt * (pitch >> 7) + slice) * 1024 + (c >> 7) * 512 + (c % 32) * 16 +
                                     ((c % 128) / 32) * 4) = words[q];
    }
}

}  // namespace

// Weight scales of a GEMM with E experts, n_feat output features and a contraction of k: stored twice, in the tiling of
// the single-CTA kernel, then in that of the CTA-pair kernel.
size_t mx_w_scale_single_bytes(int E, int n_feat, int k) { return (size_t)E * (n_feat / 128) * (k / 128) * 512; }
size_t mx_w_scale_bytes(int E, int n_feat, int k) {
    return mx_w_scale_single_bytes(E, n_feat, k) + (size_t)E * ((n_feat + MXP_NT - 1) / MXP_NT) * (k / 128) * 1024;
}

static unsigned mx_row_quantiser_blocks(long long units) {
    long long blocks = (units + 63) / 64;   // 8 warps x 8 units per block and pass
    const long long cap = (long long)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    return (unsigned)(blocks < 1 ? 1 : blocks);
}

int launch_mx_quantize_rows(long long rows, int n, const bf16* x, uint8_t* codes, uint8_t* scales, cudaStream_t s) {
    mx_quantize_rows_kernel<false><<<mx_row_quantiser_blocks(rows * (n / 128)), 256, 0, s>>>(
        reinterpret_cast<const uint4*>(x), rows, n, 0, n / 128, 0, reinterpret_cast<uint2*>(codes), scales, nullptr);
    return check_launch();
}

// w [E, k, n] -> rows [n_off, n_off + n) of the transposed codes [E, n_total, k] and the matching scale bytes
int launch_mx_quantize_w_transposed(int E, int k, int n, int n_total, int n_off, const bf16* w, uint8_t* codes_t, uint8_t* scales,
                                    cudaStream_t s) {
    const long long total = (long long)E * (k / 32) * n;
    mx_quantize_w_transposed_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        w, E, k, n, n_total, n_off, codes_t, scales, scales + mx_w_scale_single_bytes(E, n_total, k));
    return check_launch();
}

int launch_mx_swiglu_quantize(long long rows, int I, const bf16* gu, bf16* h_act, uint8_t* codes, uint8_t* scales, cudaStream_t s) {
    const long long units = rows * (I / 128);
    long long blocks = (units + 15) / 16;   // 8 warps x 2 units per block and pass
    const long long cap = (long long)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    mx_swiglu_quantize_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const uint4*>(gu), rows, I,
                                                             reinterpret_cast<uint4*>(h_act), reinterpret_cast<uint2*>(codes),
                                                             reinterpret_cast<uint32_t*>(scales));
    return check_launch();
}

int launch_mx_swiglu_bwd_quantize(long long rows, int I, const bf16* dh_act, const bf16* gu, bf16* dgu, uint8_t* codes,
                                  uint8_t* scales, cudaStream_t s) {
    const long long total = rows * (I / 8);
    mx_swiglu_bwd_quantize_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        reinterpret_cast<const uint4*>(dh_act), reinterpret_cast<const uint4*>(gu), rows, I, reinterpret_cast<uint4*>(dgu),
        reinterpret_cast<uint2*>(codes), reinterpret_cast<uint32_t*>(scales));
    return check_launch();
}

// w [E * n_feat, k] -> columns [k_off, k_off + k) of the codes [E * n_feat, k_total] and the matching scale slices
int launch_mx_quantize_w_rows(int E, int n_feat, int k, int k_total, int k_off, const bf16* w, uint8_t* codes, uint8_t* scales,
                              cudaStream_t s) {
    const long long rows = (long long)E * n_feat;
    mx_quantize_rows_kernel<true><<<mx_row_quantiser_blocks(rows * (k / 128)), 256, 0, s>>>(
        reinterpret_cast<const uint4*>(w), rows, k, n_feat, k_total / 128, k_off / 128, reinterpret_cast<uint2*>(codes), scales,
        scales + mx_w_scale_single_bytes(E, n_feat, k_total));
    return check_launch();
}

// ---- weight-gradient operands and GEMM ----
constexpr size_t MX_TOKENS_HEADER_BYTES = 8192;   // slice_prefix[E + 1] at the head of a token-quantised operand's scales
long long mx_tokens_pitch(long long R, int E) { return ((R + 127) / 128) * 128 + 128ll * E; }
size_t mx_tokens_scale_bytes(long long R, int E, int n) {
    const long long slices = mx_tokens_pitch(R, E) / 128;
    return MX_TOKENS_HEADER_BYTES + (size_t)slices * n * 4 + (size_t)((n + MXP_NT - 1) / MXP_NT) * slices * 1024;
}

int launch_mx_quantize_tokens(long long R, int E, const bf16* x, long long ld, int col0, int n, const int32_t* offsets,
                              uint8_t* codes_t, uint8_t* scales, cudaStream_t s) {
    const long long pitch = mx_tokens_pitch(R, E);
    int32_t* sp = reinterpret_cast<int32_t*>(scales);
    uint8_t* sa = scales + MX_TOKENS_HEADER_BYTES;
    uint8_t* sb = sa + (size_t)(pitch / 128) * n * 4;
    mx_slice_prefix_kernel<<<1, 1024, 0, s>>>(offsets, E, sp);
    int st_ = check_launch();
    if (st_ != MOE_OK) return st_;
    const long long total = (pitch / 128) * (n / 8);
    mx_quantize_tokens_kernel<<<(unsigned)((total + 127) / 128), 128, 0, s>>>(x, ld, col0, n, offsets, sp, E, pitch, codes_t, sa, sb);
    return check_launch();
}

// dW [E, M, N] = Q(A)^T Q(B) per expert: a_* the M-side operand ([M, pitch] codes, scales with header and words),
// b_* the N-side operand ([N, pitch] codes, its scales' pair-tiled blocks are used)
int launch_mx_wgrad(long long R, int E, int M, int N, const uint8_t* a_codes_t, const uint8_t* a_scales, const uint8_t* b_codes_t,
                    const uint8_t* b_scales, bf16* dw, cudaStream_t s) {
    const long long pitch = mx_tokens_pitch(R, E);
    const int n_slices = (int)(pitch / 128);
    const int n_tiles = (N + MXP_NT - 1) / MXP_NT, m_tiles = (M + MXP_ROWS - 1) / MXP_ROWS;
    const uint8_t* b_atoms = b_scales + MX_TOKENS_HEADER_BYTES + (size_t)n_slices * N * 4;
    CUtensorMap a, b, sfb, o;
    if (!make_map_typed(&a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes_t, (uint64_t)pitch, (uint64_t)M, MX_BK, MX_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes_t, (uint64_t)pitch, (uint64_t)N, MX_BK, MXP_NT / 2,
                        CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&sfb, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, b_atoms, 256, (uint64_t)n_tiles * n_slices, 256, 1,
                        CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_out_map(&o, dw, N, (uint64_t)E * M))
        return MOE_ERR_CUDA;
    MxPairParams p = {};
    p.prefix = reinterpret_cast<const int32_t*>(a_scales); p.E = E; p.M = M; p.m_tiles = m_tiles; p.n_tiles = n_tiles;
    p.n_cols = N; p.n_slices = n_slices; p.sa_rows = M;
    p.sa = reinterpret_cast<const uint32_t*>(a_scales + MX_TOKENS_HEADER_BYTES); p.out = dw; p.ldo = N;
    static int grid_of_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(MXP_THREADS);
    cfg.dynamicSmemBytes = MXP_SMEM_BYTES;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (grid_of_device[dev] == 0) {
        if (cudaFuncSetAttribute(mx_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, MXP_SMEM_BYTES) != cudaSuccess)
            return MOE_ERR_CUDA;
        const int sms = sm_count();
        if (sms <= 0) return MOE_ERR_CUDA;
        cfg.gridDim = dim3(2 * (sms / 2));
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, mx_pair_kernel<true>, &cfg) != cudaSuccess || clusters <= 0) return MOE_ERR_CUDA;
        if (clusters > sms / 2) clusters = sms / 2;
        grid_of_device[dev] = 2 * clusters;
    }
    cfg.gridDim = dim3(grid_of_device[dev]);
    cfg.stream = s;
    if (cudaLaunchKernelEx(&cfg, mx_pair_kernel<true>, a, b, sfb, o, p) != cudaSuccess) return MOE_ERR_CUDA;
    return check_launch();
}

// CTA pairs from this many rows per expert on average (below it the 256-row tiles are mostly padding)
constexpr long long kMxPairRows = 256;

static int launch_mx_gemm_pair(long long R, int E, int n_feat, int k, const uint8_t* a_codes, const uint8_t* a_scales,
                               const uint8_t* b_codes, const uint8_t* b_scales_pair, const int32_t* offsets, bf16* out,
                               cudaStream_t s) {
    const int n_tiles = (n_feat + MXP_NT - 1) / MXP_NT, k_tiles = k / MX_BK;
    CUtensorMap a, b, sfb, o;
    if (!make_map_typed(&a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes, k, (uint64_t)R, MX_BK, MX_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes, k, (uint64_t)E * n_feat, MX_BK, MXP_NT / 2,
                        CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&sfb, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, b_scales_pair, 256, (uint64_t)E * n_tiles * k_tiles, 256, 1,
                        CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_out_map(&o, out, n_feat, (uint64_t)R))
        return MOE_ERR_CUDA;
    MxPairParams p = {};
    p.prefix = offsets; p.E = E; p.k_tiles = k_tiles; p.n_tiles = n_tiles; p.n_cols = n_feat; p.sa_rows = R;
    p.sa = reinterpret_cast<const uint32_t*>(a_scales); p.out = out; p.ldo = n_feat;
    static int grid_of_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(MXP_THREADS);
    cfg.dynamicSmemBytes = MXP_SMEM_BYTES;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (grid_of_device[dev] == 0) {
        if (cudaFuncSetAttribute(mx_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, MXP_SMEM_BYTES) != cudaSuccess)
            return MOE_ERR_CUDA;
        const int sms = sm_count();
        if (sms <= 0) return MOE_ERR_CUDA;
        // as many pairs as can be resident at once: a pair that had to wait for a free SM pair would double the duration
        cfg.gridDim = dim3(2 * (sms / 2));
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, mx_pair_kernel<false>, &cfg) != cudaSuccess || clusters <= 0) return MOE_ERR_CUDA;
        if (clusters > sms / 2) clusters = sms / 2;
        grid_of_device[dev] = 2 * clusters;
    }
    cfg.gridDim = dim3(grid_of_device[dev]);
    cfg.stream = s;
    if (cudaLaunchKernelEx(&cfg, mx_pair_kernel<false>, a, b, sfb, o, p) != cudaSuccess) return MOE_ERR_CUDA;
    return check_launch();
}

// out[r, :] = dequant(a row r) . dequant(b[e])^T for the rows r of expert e: a [R, k] codes with scale words
// [k/128][R], b [E, n_feat, k] codes with both scale tilings, out [R, n_feat] bf16.
int launch_mx_gemm(long long R, int E, int n_feat, int k, const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                   const uint8_t* b_scales, const int32_t* offsets, bf16* out, cudaStream_t s) {
    if (R >= kMxPairRows * E)
        return launch_mx_gemm_pair(R, E, n_feat, k, a_codes, a_scales, b_codes, b_scales + mx_w_scale_single_bytes(E, n_feat, k),
                                   offsets, out, s);
    CUtensorMap a, b, o;
    if (!make_map_typed(&a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes, k, (uint64_t)R, MX_BK, MX_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_typed(&b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes, k, (uint64_t)E * n_feat, MX_BK, MX_BN,
                        CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_out_map(&o, out, n_feat, (uint64_t)R))
        return MOE_ERR_CUDA;
    MxParams p = {};
    p.offsets = offsets; p.E = E; p.k_tiles = k / MX_BK; p.n_tiles = n_feat / MX_BN; p.n_cols = n_feat; p.R = R;
    p.sa = reinterpret_cast<const uint32_t*>(a_scales); p.sb = b_scales; p.out = out; p.ldo = n_feat;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(mx_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MX_SMEM_BYTES) != cudaSuccess)
            return MOE_ERR_CUDA;
        attr_set[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return MOE_ERR_CUDA;
    mx_gemm_kernel<<<sms, MX_THREADS, MX_SMEM_BYTES, s>>>(a, b, o, p);
    return check_launch();
}

}  // namespace moe
