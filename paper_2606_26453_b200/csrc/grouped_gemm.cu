// Grouped GEMMs of the MoE layer as persistent, warp-specialised tcgen05 kernels for sm_100a.
//
// One CTA per SM walks a tile list that every CTA derives by itself from the per-expert offsets
// (no host round trip, no extra launch).  Per CTA:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 64-wide K blocks of A and B into a
//               ring of 128-byte-swizzled shared-memory stages, completion on mbarriers
//   warp 1      MMA issuer: one lane issues tcgen05.mma (bf16 -> fp32) with the accumulator in
//               tensor memory; tcgen05.commit releases ring stages and publishes finished
//               accumulators
//   warps 2..9  epilogue: tcgen05.ld the accumulator (32-lane quarter x half of the columns), apply
//               the epilogue (plain / SwiGLU), round to bf16, stage 32x32 blocks in swizzled shared
//               memory and write them with bulk tensor stores
//   warp 10     (WGRAD only) tail-fix warp: clears the surplus rows of an expert's ragged last K block once its
//               loads have landed and only then signals that stage as full, so that the MMA warp's issue
//               loop carries no tail handling (all other stages go from the loads straight to the MMA warp)
// The accumulator is double buffered (2 x 256 of the 512 TMEM columns) so the epilogue of one tile
// overlaps the main loop of the next.
//
// Two launch shapes of the same kernel:
//   single  one CTA computes a 128 x 256 tile (tcgen05.mma.cta_group::1, 4 stages of 48 KB).
//   pair    a cluster of two CTAs computes a 256 x 256 tile with tcgen05.mma.cta_group::2: each CTA
//           loads its 128 rows of A and HALF of B (6 stages of 32 KB), the tensor cores of both SMs
//           read both halves.  That cuts the bytes each SM must pull from L2 per flop by a third
//           and deepens the ring, which is what the L2 -> SM path needs at full MMA rate.  Every
//           TMA load has a single destination CTA (no multicast), but both CTAs' loads of a stage
//           report their bytes to the SAME barrier, the one of the first CTA whose MMA warp waits on
//           it (cp.async.bulk.tensor with .cta_group::2 may complete on the peer's barrier), so a
//           stage goes from the two producers to the MMA warp without a relay in between; the MMA
//           warp releases stages / publishes accumulators in both CTAs with one tcgen05.commit
//           that arrives on the barriers of both CTAs.
//
// Two ragged shapes occur:
//   row-ragged (forward, dgrad): output rows are the packed rows of an expert.  A tile starts at
//     offsets[e] + TILE_M*i; loading past the expert's last row is harmless, stores are clipped.
//     With small experts the padding of the fixed-height tiles is a sizeable share of the tensor
//     work; two pair variants avoid it: the swapped kinds (FWD_PLAIN_T, DGRAD_T: weights on the M
//     side of the MMA, the expert's rows on the N side, any tile height that is a multiple of 16)
//     and, for the SwiGLU forward, half-height last tiles (FWD_SWIGLU_H: M = 128 over the pair).
//   contraction-ragged (wgrad; the paper's dW1_e = X_e^T G_e): the expert's rows are the
//     contraction.  The last K block issues only ceil(rem/16) MMAs (guard predicates) and the < 16
//     surplus rows are zeroed in shared memory first, by the tail-fix warp of each CTA (warp 10 in the
//     first, warp 1 in the second); an expert without rows gets a zero tile.
//
// All waits are bounded: a wait that runs out records MOE_ERR_TIMEOUT in the device status word,
// raises a CTA-wide abort flag and every role leaves through the common teardown.
#include "tc_ptx.cuh"

namespace moe {

__device__ int g_device_status = 0;

#ifdef MOE_TEST_HOOKS
// Test-only build: when set, every producer leaves out the loads AND the barrier arrival of its first ring stage, so
// that the MMA warp's bounded wait on that stage runs out -- the one way to exercise the give-up path (status word,
// abort flag, teardown) without a fault, a trap or an endless loop.
__device__ int g_test_withhold_first_stage = 0;
extern "C" int moe_test_withhold_first_stage(int on) {
    return cudaMemcpyToSymbol(g_test_withhold_first_stage, &on, sizeof(int)) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
#endif

int read_and_clear_device_status(int* status_out) {
    int v = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return MOE_ERR_CUDA;
    int m = 0, x = 0;
    if (movement_read_and_clear_status(&m) != MOE_OK || mx_read_and_clear_status(&x) != MOE_OK) return MOE_ERR_CUDA;
    *status_out = v != 0 ? v : (m != 0 ? m : x);
    return MOE_OK;
}

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int CHUNK_BYTES = 64 * BK * 2;   // one 64-wide MN-major block: 64 k-rows x 128 B = 8 KB
constexpr int NUM_EPI_WARPS = 8;
constexpr int STAGING_BLOCK_BYTES = 32 * 32 * 2;   // one 32 x 32 bf16 output block
constexpr int MAX_E = 1024;
constexpr int MAX_STAGES = 6;
constexpr int NUM_THREADS = 352;   // producer warp, MMA warp, 8 epilogue warps, tail-fix warp (WGRAD)
constexpr int FIX_WARP = 2 + NUM_EPI_WARPS;
constexpr int TMEM_COLS = 512;

// The _T kinds compute the same products as FWD_PLAIN / DGRAD with the operand roles swapped: the weights are the
// M side of the MMA (128 output features per tile) and the expert's packed rows the N side, so a row tile can have
// any height that is a multiple of 16 (up to 256) instead of a fixed 128 / 256: an expert's rows are split into
// equal tiles and almost no tensor work goes to padding.  The accumulator comes out transposed (lane = feature,
// column = row); the epilogue transposes it back through its shared-memory staging blocks.
// FWD_SWIGLU_H is FWD_SWIGLU in pair mode with half-height last tiles (small experts); a kind of its own so that the
// kernel for large experts carries none of its bookkeeping.
// DGRAD_SB / DGRAD_T_SB are DGRAD / DGRAD_T of the down projection with the SwiGLU backward fused into the epilogue:
// the accumulator (dHact, fp32, never rounded) meets the saved pre-activations [g | u], which the epilogue warps fetch
// as 32 x 32 blocks with bulk tensor loads, and the kernel writes dGU = [dg | du] instead of dHact.
enum Kind { FWD_SWIGLU = 0, FWD_PLAIN = 1, DGRAD = 2, WGRAD = 3, FWD_PLAIN_T = 4, DGRAD_T = 5, FWD_SWIGLU_H = 6,
            DGRAD_SB = 7, DGRAD_T_SB = 8 };
__host__ __device__ constexpr bool wgrad(int kind) { return kind == WGRAD; }
__host__ __device__ constexpr bool swiglu(int kind) { return kind == FWD_SWIGLU || kind == FWD_SWIGLU_H; }
__host__ __device__ constexpr bool swapped(int kind) { return kind == FWD_PLAIN_T || kind == DGRAD_T || kind == DGRAD_T_SB; }
__host__ __device__ constexpr bool fused_sb(int kind) { return kind == DGRAD_SB || kind == DGRAD_T_SB; }
// the kind whose operand loads and MMAs a kind shares
__host__ __device__ constexpr int load_kind(int kind) { return kind == DGRAD_SB ? DGRAD : (kind == DGRAD_T_SB ? DGRAD_T : kind); }
constexpr int SWAP_ROWS = 256;   // most rows of a swapped tile
constexpr int SWAP_FEATS = 128;  // output features of a swapped tile

struct Params {
    const int32_t* offsets;
    int E;
    int k_blocks;        // row-ragged kinds: contraction length / 64
    int k_split;         // DGRAD: k blocks taken from the first B tensor (then the second); else k_blocks
    int n_tiles;         // output column tiles
    int m_tiles;         // WGRAD: output row tiles (of TILE_M rows) per expert
    int m_rows;          // WGRAD: output rows per expert (M)
    int n_cols;          // valid output columns (row-ragged) / total N (WGRAD)
    int b_rows_per_e;    // rows per expert in B's 2-D view
    int n_split;         // columns >= n_split go to the second output
    long long ldo;       // output row pitch (elements)
    bf16* out0;
    bf16* out1;
    bf16* gu;            // FWD_SWIGLU: [R, 2I] or null
    int I;               // FWD_SWIGLU
};

struct SharedCtl {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long landed[MAX_STAGES];   // WGRAD, MMA-issuing CTA: the stage's loads have arrived (not yet tail-fixed)
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    uint32_t tmem_base;
    int abort_flag;
    unsigned long long gu_full[NUM_EPI_WARPS];   // fused SwiGLU backward: an epilogue warp's [g | u] blocks have landed
    int stage_half[MAX_STAGES];   // FWD_SWIGLU pair: the stage belongs to a half-height tile (published by the producer)
    int stage_n[MAX_STAGES];   // swapped kinds: MMA N (rows of the tile rounded up to 16) of the tile a stage belongs to
    int32_t offs[MAX_E + 1];
    int32_t tile_prefix[MAX_E + 1];
    int32_t sorted_rows[MAX_E];   // WGRAD: row count of the expert at each position of the largest-first order
};

// Ring geometry of the two launch shapes.  WIDE: the epilogue warps also hold two 32 x 32 input blocks each (fused
// SwiGLU backward), paid for with one ring stage.
template <bool PAIR, bool WIDE = false>
struct Geo {
    static constexpr int STAGES = PAIR ? (WIDE ? 5 : 6) : 4;
    static constexpr int STAGING_BLOCKS = WIDE ? 3 : 1;   // per epilogue warp: the staging block (+ the g and u input blocks)
    static constexpr int TILE_M = PAIR ? 2 * BM : BM;        // output rows per tile (whole pair)
    static constexpr int BN_LOCAL = PAIR ? BN / 2 : BN;      // B columns this CTA keeps in shared memory
    static constexpr int A_BYTES = BM * BK * 2;              // 16 KB
    static constexpr int B_BYTES = BN_LOCAL * BK * 2;        // 16 / 32 KB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;    // 32 / 48 KB
    static constexpr int RING_BYTES = STAGES * STAGE_BYTES;  // 160 ... 192 KB
    static constexpr int STAGING_BYTES = NUM_EPI_WARPS * STAGING_BLOCKS * STAGING_BLOCK_BYTES;   // 16 KB (48 KB wide)
    static constexpr int SMEM_BYTES = RING_BYTES + STAGING_BYTES + 1024 + (int)sizeof(SharedCtl);
};

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return mbar_wait_status(bar, parity, abort_flag, &g_device_status);
}

// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 version field set.
//   K-major tile  [rows][64 k]  : 8-row groups 1024 B apart (stride byte offset); leading offset unused (1)
//   MN-major tile [chunk][64 k-rows][64 mn]: 8-k-row groups 1024 B apart (stride byte offset),
//                 64-wide mn chunks CHUNK_BYTES apart (leading byte offset)
template <bool MN_MAJOR>
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
    const uint64_t lbo = MN_MAJOR ? (uint64_t)(CHUNK_BYTES >> 4) : 1ull;
    const uint64_t sbo = 1024 >> 4;
    return (uint64_t)((addr >> 4) & 0x3FFF) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, given M (128, or 256 over a CTA pair), N and
// operand major-ness.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---- tile list ------------------------------------------------------------------------------------
struct Tile {
    int e;        // expert
    int row0;     // row-ragged: first packed row of the tile; WGRAD: first output row (m)
    int row_end;  // row-ragged: offsets[e+1]
    int n0;       // first output column
    int k_blocks; // contraction blocks of this tile
    int k_row0;   // WGRAD: first packed row of the contraction
    int k_rows;   // WGRAD: rows of the contraction
    int rows;     // swapped kinds: rows of this tile (1..256)
    int half;     // FWD_SWIGLU pair: the tile holds <= 128 rows and runs as a 128-row pair tile (64 rows per CTA)
};

// Order of an expert's m_tiles x n_tiles output tiles: bands of RASTER_BAND row tiles; inside a band
// column tile major, row tile minor.  The CTAs that run at the same time (consecutive tile ids) then
// touch about RASTER_BAND row-tile operands and gridDim/RASTER_BAND column-tile operands, a working
// set of a few tens of MB that stays in L2 whatever the expert's size.
constexpr int RASTER_BAND = 16;
__device__ __forceinline__ void raster(int local, int m_tiles, int n_tiles, int& mt, int& nt) {
    const int band = local / (RASTER_BAND * n_tiles);
    const int m0 = band * RASTER_BAND;
    const int rows = min(RASTER_BAND, m_tiles - m0);
    const int in_band = local - band * RASTER_BAND * n_tiles;
    nt = in_band / rows;
    mt = m0 + (in_band - nt * rows);
}

// The it-th tile of the CTA (pair) with index `who` out of `n_who`, or -1 when it has no more tiles.
// Row-ragged kinds: all tiles cost the same -> plain striding.  WGRAD: a tile's cost is its expert's row
// count, so experts are walked largest first and the tile sequence is dealt out boustrophedon (left to
// right on even laps, right to left on odd ones); every CTA then gets within ~1 % of the same number of
// contraction blocks even under heavy routing imbalance (plain striding: up to 11 % off on the skewed
// workloads).
template <int KIND>
__device__ __forceinline__ long long tile_of(long long it, long long who, long long n_who, long long total) {
    long long t;
    if (wgrad(KIND)) {
        if (it * n_who >= total) return -1;
        t = it * n_who + ((it & 1) ? n_who - 1 - who : who);
    } else {
        t = who + it * n_who;
    }
    return t < total ? t : -1;
}

template <int KIND>
__device__ __forceinline__ long long total_tiles(const Params& p, const SharedCtl* ctl) {
    if (wgrad(KIND)) return (long long)p.E * p.m_tiles * p.n_tiles;
    return (long long)ctl->tile_prefix[p.E] * p.n_tiles;
}

template <int KIND, int TILE_M>
__device__ __forceinline__ Tile decode_tile(const Params& p, const SharedCtl* ctl, long long t) {
    Tile tl;
    if (wgrad(KIND)) {
        const int per_e = p.m_tiles * p.n_tiles;
        const int e_rank = (int)(t / per_e);
        tl.e = ctl->tile_prefix[e_rank];   // WGRAD: this array holds the experts ordered by row count, largest first
        const int local = (int)(t - (long long)e_rank * per_e);
        int mt, nt;
        raster(local, p.m_tiles, p.n_tiles, mt, nt);
        tl.row0 = mt * TILE_M;
        tl.n0 = nt * BN;
        tl.k_row0 = ctl->offs[tl.e];
        tl.k_rows = ctl->offs[tl.e + 1] - tl.k_row0;
        tl.k_blocks = (tl.k_rows + BK - 1) / BK;
        tl.row_end = 0;
        tl.rows = 0;
        tl.half = 0;
    } else {
        // tile_prefix[e] = number of TILE_M-row tiles of experts < e
        int lo = 0, hi = p.E;                          // largest e with tile_prefix[e]*n_tiles <= t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((long long)ctl->tile_prefix[mid] * p.n_tiles <= t) lo = mid; else hi = mid;
        }
        tl.e = lo;
        const int m_tiles_e = ctl->tile_prefix[lo + 1] - ctl->tile_prefix[lo];
        const int local = (int)(t - (long long)ctl->tile_prefix[lo] * p.n_tiles);
        int mt, nt;
        raster(local, m_tiles_e, p.n_tiles, mt, nt);
        tl.row_end = ctl->offs[lo + 1];
        tl.rows = 0;
        if (swapped(KIND)) {
            // the expert's rows in m_tiles_e equal tiles, each a multiple of 16 rows (the last one takes what is left)
            const int n_e = tl.row_end - ctl->offs[lo];
            const int per_tile = ((n_e + m_tiles_e - 1) / m_tiles_e + 15) & ~15;
            tl.row0 = ctl->offs[lo] + mt * per_tile;
            tl.rows = min(per_tile, tl.row_end - tl.row0);
            tl.n0 = nt * TILE_M;   // output features per tile: 128, or 256 over a CTA pair
        } else {
            tl.row0 = ctl->offs[lo] + mt * TILE_M;
            tl.n0 = nt * BN;
        }
        tl.half = (KIND == FWD_SWIGLU_H && tl.row_end - tl.row0 <= BM) ? 1 : 0;
        tl.k_blocks = p.k_blocks;
        tl.k_row0 = 0;
        tl.k_rows = 0;
    }
    return tl;
}

// WGRAD: clear contraction rows [z0, z1) of a stage (A chunks and this CTA's B chunks are contiguous)
__device__ __forceinline__ void zero_k_rows(uint8_t* stage_ptr, int n_chunks, int z0, int z1, int lane) {
    const int per_row = n_chunks * 8;   // 16-byte pieces per k-row over all chunks
    for (int i = lane; i < (z1 - z0) * per_row; i += 32) {
        const int r = z0 + i / per_row, q = i % per_row;
        const int chunk = q >> 3, piece = q & 7;
        *reinterpret_cast<uint4*>(stage_ptr + chunk * CHUNK_BYTES + r * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// The TMA loads of one ring stage: k-block `kb` of tile `tl`, for the CTA with row offset `my_rows` inside
// the tile (and, in pair mode, its half of B).  (Prefetching the same boxes into L2 a few k-blocks ahead was
// tried and cost 10-15 %: the L2 -> SM path, not DRAM latency, is what these kernels saturate.)
// `full` is the barrier the loads report to: a shared::cta address, or (REMOTE_BAR, pair mode) a shared::cluster address
// of a barrier of the MMA-issuing CTA.
template <int KIND, bool PAIR, bool REMOTE_BAR>
__device__ __forceinline__ void stage_loads(const Tile& tl, int kb, const Params& p, const CUtensorMap* map_a,
                                         const CUtensorMap* map_r2, const CUtensorMap* map_r1,
                                         const CUtensorMap* map_b0, const CUtensorMap* map_b1, uint32_t a_dst,
                                         uint32_t b_dst, uint32_t full, uint32_t rank, int my_rows) {
    auto tma_load_2d = [](uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
        if (REMOTE_BAR) tma_load_2d_pair(dst, map, x, y, bar); else moe::tma_load_2d(dst, map, x, y, bar);
    };
    auto tma_load_3d = [](uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
        if (REMOTE_BAR) tma_load_3d_pair(dst, map, x, y, z, bar); else moe::tma_load_3d(dst, map, x, y, z, bar);
    };
    const int n_local = tl.n0 + (PAIR ? my_rows : 0);   // first B column this CTA loads
    if (swapped(KIND)) {
        // M side (a_dst): the weight tile, 128 output features x 64 k.  N side (b_dst): the tile's rows in boxes of
        // 64 rows (map_a is the activation map with a 64-row box), only as many boxes as the tile has rows.
        // In pair mode each CTA loads its own 128 features and half of the tile's rows (N/2 of the MMA's N,
        // N = rows rounded up to 16), in boxes of 32 rows; a single CTA loads all rows in boxes of 64.
        const int feat0 = tl.n0 + (PAIR ? (int)rank * SWAP_FEATS : 0);
        if (KIND == FWD_PLAIN_T) {
            tma_load_3d(a_dst, map_b0, 0, tl.e * p.b_rows_per_e + kb * BK, feat0 >> 6, full);
        } else {
            const bool second = kb >= p.k_split;
            const int kx = (second ? kb - p.k_split : kb) * BK;
            tma_load_2d(a_dst, second ? map_b1 : map_b0, kx, tl.e * p.b_rows_per_e + feat0, full);
        }
        // at most two loads: boxes of 1, 2 or 4 times BOX rows (map_r1, map_r2, map_a), or 2 + 1
        constexpr int BOX = PAIR ? 32 : 64;
        const int my_n = PAIR ? (((tl.rows + 15) & ~15) >> 1) : tl.rows;           // rows this CTA provides
        const int my_row0 = tl.row0 + (PAIR ? (int)rank * my_n : 0);
        if (my_n <= BOX) {
            tma_load_2d(b_dst, map_r1, kb * BK, my_row0, full);
        } else if (my_n <= 2 * BOX) {
            tma_load_2d(b_dst, map_r2, kb * BK, my_row0, full);
        } else if (my_n <= 3 * BOX) {
            tma_load_2d(b_dst, map_r2, kb * BK, my_row0, full);
            tma_load_2d(b_dst + 2 * BOX * 128, map_r1, kb * BK, my_row0 + 2 * BOX, full);
        } else {
            tma_load_2d(b_dst, map_a, kb * BK, my_row0, full);
        }
    } else if (wgrad(KIND)) {
        const int krow = tl.k_row0 + kb * BK;
        // MN-major operands: one 3-D box = all 64-wide chunks, chunk-major in shared memory
        tma_load_3d(a_dst, map_a, 0, krow, (tl.row0 + my_rows) >> 6, full);
        tma_load_3d(b_dst, map_b0, 0, krow, n_local >> 6, full);
    } else {
        // half-height pair tile (FWD_SWIGLU): rows [row0, row0+64) in the first CTA, [row0+64, row0+128) in the second;
        // map_r1 is the A map with a 64-row box there
        if (KIND == FWD_SWIGLU_H && tl.half) tma_load_2d(a_dst, map_r1, kb * BK, tl.row0 + (int)rank * (BM / 2), full);
        else tma_load_2d(a_dst, map_a, kb * BK, tl.row0 + my_rows, full);
        if (load_kind(KIND) == DGRAD) {
            const bool second = kb >= p.k_split;
            const int kx = (second ? kb - p.k_split : kb) * BK;
            tma_load_2d(b_dst, second ? map_b1 : map_b0, kx, tl.e * p.b_rows_per_e + n_local, full);
        } else if (KIND == FWD_PLAIN) {
            const int ky = tl.e * p.b_rows_per_e + kb * BK;
            tma_load_3d(b_dst, map_b0, 0, ky, n_local >> 6, full);
        } else {  // FWD_SWIGLU: 128 gate columns then 128 up columns
            const int ky = tl.e * p.b_rows_per_e + kb * BK;
            const int ng = tl.n0 >> 1;   // n0 counts fused (gate+up) columns
            if (PAIR) {
                // pair mode with half-height tiles (small experts): the maps have one-chunk (64-column) boxes.  Full tile: the first CTA holds the 128 gate
                // columns of B, the second the 128 up columns.  Half tile: the accumulator of an M = 128 pair MMA
                // keeps columns 0..127 in lanes 0..63 and columns 128..255 in lanes 64..127, and gate and up of a
                // feature must meet in one lane: each CTA holds [64 gate | 64 up] columns of the same 64 features.
                const int c = ng >> 6;
                const CUtensorMap* mb = rank == 0 ? map_b0 : map_b1;
                if (KIND != FWD_SWIGLU_H) {   // large experts: two-chunk boxes, one load
                    tma_load_3d(b_dst, mb, 0, ky, c, full);
                } else if (tl.half) {
                    tma_load_3d(b_dst, map_b0, 0, ky, c + (int)rank, full);
                    tma_load_3d(b_dst + CHUNK_BYTES, map_b1, 0, ky, c + (int)rank, full);
                } else {
                    tma_load_3d(b_dst, mb, 0, ky, c, full);
                    tma_load_3d(b_dst + CHUNK_BYTES, mb, 0, ky, c + 1, full);
                }
            } else {
                tma_load_3d(b_dst, map_b0, 0, ky, ng >> 6, full);
                tma_load_3d(b_dst + 2 * CHUNK_BYTES, map_b1, 0, ky, ng >> 6, full);
            }
        }
    }
}

// ---- the kernel -----------------------------------------------------------------------------------
// Operand major-ness per kind:
//   FWD_*  : A K-major (activations [R, K]),   B MN-major (weights [E*K, N], N contiguous)
//   DGRAD  : A K-major,                        B K-major  (weights [E*N, K], K contiguous)
//   WGRAD  : A MN-major (activations [R, M]),  B MN-major (gradients [R, N])
template <int KIND, bool PAIR>
__global__ void __launch_bounds__(NUM_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
                    const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_o0,
                    const __grid_constant__ CUtensorMap map_o1, const __grid_constant__ CUtensorMap map_x,
                    const Params p) {
    using G = Geo<PAIR, fused_sb(KIND)>;
    constexpr int STAGES = G::STAGES;
    constexpr int STAGE_BYTES = G::STAGE_BYTES;
    constexpr bool SWAP = swapped(KIND);
    // SwiGLU forward in pair mode: an expert's last <= 128 rows run as a half-height tile (tcgen05.mma M = 128 over the
    // pair, 64 rows per CTA, half the MMA time) instead of a padded 256-row tile
    constexpr bool HALF_TILES = (KIND == FWD_SWIGLU_H);
    static_assert(!HALF_TILES || PAIR, "half-height tiles exist in pair mode only");
    constexpr int ROW_TILE = SWAP ? SWAP_ROWS : G::TILE_M;   // rows an expert's tile count is computed from
    // operand major-ness of the MMA's M side (A) and N side (B); for the swapped kinds A is the weight tile
    constexpr bool A_MN = (wgrad(KIND) || KIND == FWD_PLAIN_T);
    constexpr bool B_MN = (swiglu(KIND) || KIND == FWD_PLAIN || wgrad(KIND));
    constexpr uint32_t IDESC = make_idesc(G::TILE_M, BN, A_MN, B_MN);
    constexpr uint32_t IDESC_HALF = make_idesc(BM, BN, A_MN, B_MN);   // 128 x 256 over the CTA pair
    constexpr uint32_t A_KSTEP = A_MN ? 2048 : 32;   // bytes per 16 k inside a stage
    constexpr uint32_t B_KSTEP = B_MN ? 2048 : 32;
    constexpr int STAGE_CHUNKS = BM / 64 + G::BN_LOCAL / 64;   // 64-wide MN-major blocks per stage (WGRAD)

    extern __shared__ uint8_t smem_raw[];
    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(tiles_ptr + G::RING_BYTES + G::STAGING_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;          // 0 = the CTA that issues the MMAs
    const long long first_tile = PAIR ? (long long)(blockIdx.x >> 1) : (long long)blockIdx.x;
    const long long tile_stride = PAIR ? (long long)(gridDim.x >> 1) : (long long)gridDim.x;
    const int my_rows = rank * BM;                                 // this CTA's row offset inside the tile

    // ---- set-up: barriers, schedule tables, TMEM ----
    for (int e = threadIdx.x; e <= p.E; e += NUM_THREADS) ctl->offs[e] = p.offsets[e];
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // pair mode, first CTA: own producer's (WGRAD: own tail-fix warp's) arrive + the relay's remote arrive
            mbar_init(smem_u32(&ctl->full[s]), (PAIR && rank == 0) ? 2 : 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
            mbar_init(smem_u32(&ctl->landed[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctl->tmem_full[a]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[a]), PAIR ? 2 * NUM_EPI_WARPS : NUM_EPI_WARPS);
        }
        mbar_init(smem_u32(&ctl->drain), 1);
        for (int w = 0; w < NUM_EPI_WARPS; ++w) mbar_init(smem_u32(&ctl->gu_full[w]), 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b0);
        prefetch_tmap(&map_b1);
        prefetch_tmap(&map_o0);
        prefetch_tmap(&map_o1);
        prefetch_tmap(&map_x);
    }
    __syncthreads();
    if (wgrad(KIND)) {
        // experts by row count, largest first (ties: lower id first): rank by counting, O(E^2 / threads)
        for (int e = threadIdx.x; e < p.E; e += NUM_THREADS) {
            const int n_e = ctl->offs[e + 1] - ctl->offs[e];
            int rank = 0;
            for (int f = 0; f < p.E; ++f) {
                const int n_f = ctl->offs[f + 1] - ctl->offs[f];
                rank += (n_f > n_e || (n_f == n_e && f < e)) ? 1 : 0;
            }
            ctl->tile_prefix[rank] = e;
            ctl->sorted_rows[rank] = n_e;
        }
    } else if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < p.E; ++e) {
            ctl->tile_prefix[e] = run;
            run += (ctl->offs[e + 1] - ctl->offs[e] + ROW_TILE - 1) / ROW_TILE;
        }
        ctl->tile_prefix[p.E] = run;
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                         "r"((uint32_t)TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                         "r"((uint32_t)TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // the other CTA's barriers and tensor memory exist from here on
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const long long n_tiles_total = total_tiles<KIND>(p, ctl);

    if (warp == 0) {
        // ================= TMA producer (both CTAs of a pair; each fills its own ring) =================
        // Where a stage's loads report: normally straight to full[stage] of the MMA-issuing CTA -- in pair mode both
        // CTAs' loads complete on that one barrier (two arrivals, one per producer, each announcing its own bytes), so
        // a stage travels producer -> loads -> MMA with no relay hop.  Only a weight-gradient stage whose ragged last
        // K block needs surplus rows cleared reports to this CTA's landed[stage]; the tail-fix / relay warp clears the
        // rows and makes the arrival on full[stage] in the producer's place.
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            const uint32_t full0 = PAIR ? map_to_cta(smem_u32(&ctl->full[0]), 0) : smem_u32(&ctl->full[0]);
            for (long long it = 0; ok; ++it) {
                const long long t = tile_of<KIND>(it, first_tile, tile_stride, n_tiles_total);
                if (t < 0) break;
                const Tile tl = decode_tile<KIND, G::TILE_M>(p, ctl, t);
                for (int kb = 0; kb < tl.k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const bool fix = wgrad(KIND) && kb == tl.k_blocks - 1 && (tl.k_rows & 15) != 0;
                    uint32_t bytes = STAGE_BYTES;
                    if (SWAP) {
                        ctl->stage_n[stage] = (tl.rows + 15) & ~15;   // read by the MMA thread after its wait on full[stage]
                        const int my_n = PAIR ? (((tl.rows + 15) & ~15) >> 1) : tl.rows;
                        constexpr int BOX = PAIR ? 32 : 64;
                        bytes = G::A_BYTES + min(4, (my_n + BOX - 1) / BOX) * (BOX * BK * 2);
                    } else if (HALF_TILES) {
                        ctl->stage_half[stage] = tl.half;   // read by the MMA thread after its wait on full[stage]
                        if (tl.half) bytes = STAGE_BYTES - G::A_BYTES / 2;
                    }
                    const uint32_t a_dst = tiles_base + stage * STAGE_BYTES;
#ifdef MOE_TEST_HOOKS
                    if (g_test_withhold_first_stage != 0 && issued == 0) {
                        ++issued;
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
#endif
                    if (fix) {
                        const uint32_t land = smem_u32(&ctl->landed[stage]);
                        mbar_arrive_expect_tx(land, bytes);
                        stage_loads<KIND, PAIR, false>(tl, kb, p, &map_a, &map_o1, &map_x, &map_b0, &map_b1, a_dst, a_dst + G::A_BYTES,
                                                       land, rank, my_rows);
                    } else {
                        const uint32_t land = full0 + stage * (uint32_t)sizeof(unsigned long long);
                        if (PAIR) mbar_arrive_expect_tx_cluster(land, bytes); else mbar_arrive_expect_tx(land, bytes);
                        stage_loads<KIND, PAIR, PAIR>(tl, kb, p, &map_a, &map_o1, &map_x, &map_b0, &map_b1, a_dst, a_dst + G::A_BYTES,
                                                      land, rank, my_rows);
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok && issued != 0) {
                // leave no bulk copy in flight.  The copies report to barriers this thread cannot always poll (the other
                // CTA's), so simply outwait them: a copy that was issued completes within microseconds.
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 1 && rank == 0) {
        // ================= MMA issuer (first CTA of a pair): one thread =================
        // Measured on this part: the issuing thread spends ~85 cycles on each tcgen05.mma and the tensor pipe
        // queues about two of them, so per 64-wide K block (4 MMAs, 512 pipe cycles) the thread has only
        // ~170 cycles for everything else before the pipe runs dry; shared-memory loads and barrier polls
        // take 100+ cycles each here because TMA fills and operand reads keep the shared-memory pipe busy.
        // The role is therefore a single thread (no warp synchronisation, no divergence) whose loop holds
        // nothing but wait / MMAs / commit.  Per tile: the id and row count of the NEXT tile are fetched
        // before the K loop (the load's latency passes under the MMAs), the last block is peeled out of the
        // loop (guard predicates for the ragged last block of a WGRAD tile), and whether the next accumulator
        // buffer is free is tested, without blocking, just before that last block.
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t acc = 0, acc_phase = 0;
            bool ok = true;
            const long long per_e = (long long)p.m_tiles * p.n_tiles;   // WGRAD: tiles per expert
            int e_pos = 0;                                              // WGRAD: position in the largest-first order
            long long e_end = per_e;
            auto rows_of = [&](long long tile) -> int {                 // WGRAD; tile ids of one CTA only grow
                while (tile >= e_end) { ++e_pos; e_end += per_e; }
                return ctl->sorted_rows[e_pos];
            };
            // one K block: n_mma MMAs from ring stage `stage`, then the stage is released
            uint32_t idesc = IDESC;
            auto issue_block = [&](uint32_t d_tmem, bool first_block, int n_mma, bool partial) -> bool {
                if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag)) return false;
                tc_fence_after();
                // swapped kinds: the MMA's N is the tile's row count (rounded up to 16), published with each stage
                if (SWAP && first_block) idesc = make_idesc(G::TILE_M, ctl->stage_n[stage], A_MN, B_MN);
                if (HALF_TILES && first_block) idesc = ctl->stage_half[stage] ? IDESC_HALF : IDESC;
                const uint32_t a_base = tiles_base + stage * STAGE_BYTES;
                const uint64_t a_desc = make_smem_desc<A_MN>(a_base);
                const uint64_t b_desc = make_smem_desc<B_MN>(a_base + G::A_BYTES);
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    const uint32_t accumulate = (!first_block || kk != 0) ? 1u : 0u;
                    if (partial)
                        tc_mma_if<PAIR>(d_tmem, a_desc + (uint64_t)((kk * A_KSTEP) >> 4),
                                        b_desc + (uint64_t)((kk * B_KSTEP) >> 4), IDESC, accumulate, kk < n_mma ? 1u : 0u);
                    else
                        tc_mma<PAIR>(d_tmem, a_desc + (uint64_t)((kk * A_KSTEP) >> 4),
                                     b_desc + (uint64_t)((kk * B_KSTEP) >> 4), (SWAP || HALF_TILES) ? idesc : IDESC, accumulate);
                }
                tc_commit<PAIR>(smem_u32(&ctl->empty[stage]));
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                return true;
            };
            long long t = tile_of<KIND>(0, first_tile, tile_stride, n_tiles_total);
            int k_rows = (KIND == WGRAD && t >= 0) ? rows_of(t) : 0;
            bool acc_free = false;   // the accumulator buffer of the current tile is already known to be free
            for (long long it = 0; ok && t >= 0; ++it) {
                const long long t_next = tile_of<KIND>(it + 1, first_tile, tile_stride, n_tiles_total);
                const int k_rows_next = (KIND == WGRAD && t_next >= 0) ? rows_of(t_next) : 0;
                // whole K blocks, and MMAs of the ragged last block (WGRAD; its surplus rows were cleared
                // before full[] was signalled)
                const int n_full = (KIND == WGRAD) ? (k_rows >> 6) : p.k_blocks;
                const int n_tail = (KIND == WGRAD) ? (((k_rows & (BK - 1)) + 15) >> 4) : 0;
                if (!acc_free && !mbar_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                const int n_main = n_tail != 0 ? n_full : n_full - 1;   // blocks before the peeled last one
                for (int kb = 0; kb < n_main; ++kb)
                    if (!issue_block(d_tmem, kb == 0, BK / 16, false)) { ok = false; break; }
                if (!ok) break;
                // the next tile's accumulator buffer was handed to the epilogue one tile ago: usually free by now
                const uint32_t acc_n = acc ^ 1u, acc_phase_n = acc_phase ^ acc;
                acc_free = mbar_test_wait(smem_u32(&ctl->tmem_empty[acc_n]), acc_phase_n ^ 1u);
                if (n_main >= 0) {
                    if (n_tail != 0) { if (!issue_block(d_tmem, n_main == 0, n_tail, true)) { ok = false; break; } }
                    else             { if (!issue_block(d_tmem, n_main == 0, BK / 16, false)) { ok = false; break; } }
                }
                tc_commit<PAIR>(smem_u32(&ctl->tmem_full[acc]));
                acc = acc_n;
                acc_phase = acc_phase_n;
                t = t_next;
                k_rows = k_rows_next;
            }
        }
        __syncwarp();
        // all issued MMAs must have retired before tensor memory is released
        if (lane == 0) {
            tc_commit_local<PAIR>(smem_u32(&ctl->drain));
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < WAIT_LIMIT_NS) {}
        }
        __syncwarp();
    } else if (wgrad(KIND) && ((warp == 1 && rank != 0) || (warp == FIX_WARP && rank == 0))) {
        // ================= tail-fix warp (weight gradients): warp 10 of the MMA-issuing CTA, warp 1 of the second =======
        // Only the ragged last K block of a tile whose row count is not a multiple of 16 comes this way: its loads
        // complete on landed[stage]; this warp clears the surplus contraction rows of its CTA's half of the stage and
        // then makes this CTA's arrival on full[stage] of the MMA-issuing CTA (locally, or with a remote arrive).  All
        // other stages are skipped: it only keeps count of them.
        const bool remote = rank != 0;
        uint32_t stage = 0;
        uint32_t landed_parity = 0;   // bit s: parity of the next use of landed[s]
        bool ok = true;
        for (long long it = 0; ok; ++it) {
            const long long t = tile_of<KIND>(it, first_tile, tile_stride, n_tiles_total);
            if (t < 0) break;
            const Tile tl = decode_tile<KIND, G::TILE_M>(p, ctl, t);
            if (tl.k_blocks == 0) continue;
            const uint32_t last = (stage + (uint32_t)tl.k_blocks - 1u) % (uint32_t)STAGES;
            if ((tl.k_rows & 15) != 0) {
                if (!mbar_wait(smem_u32(&ctl->landed[last]), (landed_parity >> last) & 1u, abort_flag)) { ok = false; break; }
                landed_parity ^= 1u << last;
                const int rem = tl.k_rows - (tl.k_blocks - 1) * BK;
                zero_k_rows(tiles_ptr + last * STAGE_BYTES, STAGE_CHUNKS, rem, ((rem + 15) >> 4) * 16, lane);
                __syncwarp();
                if (lane == 0) {
                    if (remote) mbar_arrive_remote(map_to_cta(smem_u32(&ctl->full[last]), 0));
                    else mbar_arrive(smem_u32(&ctl->full[last]));
                }
            }
            stage = (last + 1u) % (uint32_t)STAGES;
        }
    } else if (warp >= 2 && warp < FIX_WARP) {
        // ================= epilogue (warps 2..9) =================
        // Each warp owns a 32-row slab (its TMEM lane quarter) and half of the tile's columns.  A
        // 32 x 32 block is rounded to bf16, written to the warp's 2 KB staging buffer in the 64-byte
        // swizzle pattern and sent to global memory by one bulk tensor store, so the LSU never issues
        // scattered global stores next to the TMA fills of the operand ring.  A slab that is only partly
        // inside its expert (row-ragged kinds) falls back to predicated 16-byte row stores.
        const int quarter = warp & 3;               // TMEM lanes [32*quarter, 32*quarter+32)
        const int half = (warp - 2) >> 2;           // which half of the tile's columns this warp handles
        uint8_t* stage_ptr = tiles_ptr + G::RING_BYTES + (warp - 2) * (G::STAGING_BLOCKS * STAGING_BLOCK_BYTES);
        const int sw = (lane >> 1) & 3;             // 64-byte swizzle: 16-byte piece j of row r sits at j ^ ((r>>1)&3)
        uint32_t n_stores = 0;                      // bulk stores issued so far by this warp

        // before the staging block is written again: all earlier stores of this warp must have read it
        auto staging_free = [&]() {
            if (n_stores != 0) {
                if (lane == 0) bulk_wait_read0();
                __syncwarp();
            }
        };
        auto send_block = [&](const CUtensorMap* map, int x, int y) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(map, x, y, smem_u32(stage_ptr));
                bulk_commit();
            }
            ++n_stores;
        };
        // stage one 32x32 bf16 block (this thread: 16 packed words of its row) and issue its bulk store
        auto stage_and_store = [&](const uint32_t (&w)[16], const CUtensorMap* map, int x, int y) {
            staging_free();
            uint8_t* my_row = stage_ptr + lane * 64;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                *reinterpret_cast<uint4*>(my_row + ((j ^ sw) << 4)) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            send_block(map, x, y);
        };
        auto direct_store = [&](const uint32_t (&w)[16], bf16* dst) {
            uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
            for (int j = 0; j < 4; ++j) d4[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        };
        // swapped kinds: this lane holds one output feature for 32 consecutive rows; the block is transposed on its
        // way into the staging buffer (row j of the block, feature `lane`: 2-byte stores, 64 contiguous bytes per
        // warp instruction) and then stored like any other 32 x 32 block
        auto stage_transposed_and_store = [&](const float (&v)[32], const CUtensorMap* map, int x, int y) {
            staging_free();
            const int piece = lane >> 3, within = (lane & 7) * 2;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                *reinterpret_cast<__nv_bfloat16*>(stage_ptr + j * 64 + (((piece ^ ((j >> 1) & 3)) << 4) + within)) =
                    __float2bfloat16_rn(v[j]);
            send_block(map, x, y);
        };
        // fused SwiGLU backward: the warp's g and u input blocks (behind its staging block), fetched with two bulk
        // tensor loads from the saved pre-activations [R, 2I] (map_b1: 32 x 32 boxes, 64-byte swizzle)
        uint8_t* g_blk = stage_ptr + STAGING_BLOCK_BYTES;
        uint8_t* u_blk = stage_ptr + 2 * STAGING_BLOCK_BYTES;
        const uint32_t gu_bar = smem_u32(&ctl->gu_full[warp - 2]);
        uint32_t gu_phase = 0;
        auto fetch_gu = [&](int x, int y) {   // x: column inside [0, I), y: first row of the block
            if (lane == 0) {
                mbar_arrive_expect_tx(gu_bar, 2 * STAGING_BLOCK_BYTES);
                tma_load_2d(smem_u32(g_blk), &map_b1, x, y, gu_bar);
                tma_load_2d(smem_u32(u_blk), &map_b1, p.I + x, y, gu_bar);
            }
        };
        // Called by every lane with a value derived from ALL of its reads of the input blocks, before the next fetch
        // into them is issued: the empty asm cannot run before those reads have delivered their data, and the warp
        // barrier then holds lane 0's fetch back until every lane got here.  (A warp barrier alone only orders the
        // ISSUE of the reads; under the operand traffic of the main loop a read can sit in the shared-memory queue long
        // enough for a bulk load that hits in L2 to overwrite its word first: seen as a few wrong elements per 10^8.)
        auto inputs_consumed = [&](uint32_t seen) {
            asm volatile("" ::"r"(seen) : "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
        };
        // dg = dh*u*s*(1+g*(1-s)), du = dh*g*s with s = 1/(1+exp(-g))
        auto swiglu_grad = [](float dh, float g, float u, float& dg, float& du) {
            const float sg = __fdividef(1.f, 1.f + __expf(-g));
            dg = dh * u * sg * (1.f + g * (1.f - sg));
            du = dh * g * sg;
        };
        // a zero tile (expert without rows, weight gradients): clear the staging block once and send it to the four
        // 32 x 32 output blocks of this warp that start at column n_first, back to back
        auto zero_blocks = [&](int n_first, int y) {
            staging_free();
#pragma unroll
            for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(stage_ptr + lane * 64 + j * 16) = make_uint4(0, 0, 0, 0);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                for (int c = 0; c < BN / 64; ++c) {
                    const int n = n_first + c * 32;
                    if (n >= p.n_cols) continue;
                    const bool first = n < p.n_split;
                    tma_store_2d(first ? &map_o0 : &map_o1, first ? n : n - p.n_split, y, smem_u32(stage_ptr));
                }
                bulk_commit();
            }
            ++n_stores;
        };
        // the warp's four 32-column blocks of one accumulator (tensor-memory address t_acc, first output column n_base):
        // software pipeline, the tensor-memory load of the next block is in flight while the current one is converted,
        // staged and stored
        auto drain_plain = [&](uint32_t t_acc, int n_base, bool have_acc, int rows_valid, int y, long long row) {
            constexpr int NC = BN / 64;
            const int c0 = half * NC;
            auto emit = [&](const uint32_t (&v)[32], int c) {
                const int n = n_base + c * 32;
                if (rows_valid == 0 || n >= p.n_cols) return;
                uint32_t w[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) w[j] = pack_bf16(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                const bool first = n < p.n_split;
                const int x = first ? n : n - p.n_split;
                if (rows_valid == 32) {
                    stage_and_store(w, first ? &map_o0 : &map_o1, x, y);
                } else if (lane < rows_valid) {
                    direct_store(w, p.out0 + row * p.ldo + x);     // row-ragged kinds have a single output
                }
            };
            uint32_t va[32], vb[32];
            if (have_acc) {
                tc_ld32(t_acc + c0 * 32, va);
            } else {   // only reached for a partial zero slab, which cannot occur; kept total
#pragma unroll
                for (int j = 0; j < 32; ++j) va[j] = vb[j] = 0u;
            }
#pragma unroll
            for (int i = 0; i < NC; i += 2) {
                if (have_acc) {
                    tc_wait_ld();
                    tc_ld32(t_acc + (c0 + i + 1) * 32, vb);
                }
                emit(va, c0 + i);
                if (have_acc) {
                    tc_wait_ld();
                    if (i + 2 < NC) tc_ld32(t_acc + (c0 + i + 2) * 32, va);
                }
                emit(vb, c0 + i + 1);
            }
        };
        const uint32_t tmem_empty_remote0 = PAIR ? map_to_cta(smem_u32(&ctl->tmem_empty[0]), 0) : 0u;
        const uint32_t tmem_empty_remote1 = PAIR ? map_to_cta(smem_u32(&ctl->tmem_empty[1]), 0) : 0u;

        uint32_t acc = 0, acc_phase = 0;
        for (long long it = 0;; ++it) {
            const long long t = tile_of<KIND>(it, first_tile, tile_stride, n_tiles_total);
            if (t < 0) break;
            const Tile tl = decode_tile<KIND, G::TILE_M>(p, ctl, t);
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(quarter * 32) << 16);
            // first row of this warp's slab.  Half-height pair tile (FWD_SWIGLU, M = 128 over two CTAs): this CTA holds
            // 64 rows; tensor-memory lanes 0..63 carry them for the MMA's columns 0..127, lanes 64..127 carry the same
            // rows for columns 128..255 (128 tensor-memory columns per accumulator instead of 256).
            const bool half_tile = HALF_TILES && tl.half;
            const int slab0 = half_tile ? tl.row0 + (int)rank * (BM / 2) + (quarter & 1) * 32 : tl.row0 + my_rows + quarter * 32;
            // rows of the slab that are owed: inside the expert (row-ragged kinds) / inside M (WGRAD); 32 = whole slab
            const int rows_valid = wgrad(KIND) ? (slab0 < p.m_rows ? 32 : 0) : max(0, min(32, tl.row_end - slab0));
            const int slab_y = wgrad(KIND) ? tl.e * p.m_rows + slab0 : slab0;
            const long long row = (long long)slab0 + lane;
            if (SWAP) {
                // lane = output feature, tensor-memory column = row of the tile; the two warps of a lane quarter
                // take the 32-row blocks alternately
                const int feat0 = tl.n0 + (PAIR ? (int)rank * SWAP_FEATS : 0) + quarter * 32;
                const int n_row_blocks = (tl.rows + 31) >> 5;
                const bool feats_owed = feat0 < p.n_cols;
                if (fused_sb(KIND) && feats_owed && half < n_row_blocks) fetch_gu(feat0, tl.row0 + half * 32);
#pragma unroll 1
                for (int i = half; i < n_row_blocks; i += 2) {
                    uint32_t vr[32];
                    tc_ld32(taddr + i * 32, vr);
                    tc_wait_ld();
                    if (!feats_owed) continue;
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(vr[j]);
                    const int r0 = tl.row0 + i * 32;
                    const int rv = min(32, tl.rows - i * 32);
                    if (fused_sb(KIND)) {
                        // element (row j, feature `lane`) of the g and u blocks; then the next block's fetch may start
                        if (!mbar_wait(gu_bar, gu_phase, abort_flag)) break;
                        gu_phase ^= 1u;
                        const int piece = lane >> 3, within = (lane & 7) * 2;
                        float du[32];
                        uint32_t seen = 0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int off = j * 64 + (((piece ^ ((j >> 1) & 3)) << 4) + within);
                            const uint32_t gr = *reinterpret_cast<const uint16_t*>(g_blk + off);
                            const uint32_t ur = *reinterpret_cast<const uint16_t*>(u_blk + off);
                            seen ^= gr ^ (ur << 16);
                            swiglu_grad(v[j], __uint_as_float(gr << 16), __uint_as_float(ur << 16), v[j], du[j]);
                        }
                        if (i + 2 < n_row_blocks) {
                            inputs_consumed(seen);   // all reads of the two input blocks have returned
                            fetch_gu(feat0, tl.row0 + (i + 2) * 32);
                        }
                        if (rv == 32) {
                            stage_transposed_and_store(v, &map_o0, feat0, r0);
                            stage_transposed_and_store(du, &map_o0, p.I + feat0, r0);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < rv) {
                                    p.out0[(long long)(r0 + j) * p.ldo + feat0 + lane] = __float2bfloat16_rn(v[j]);
                                    p.out0[(long long)(r0 + j) * p.ldo + p.I + feat0 + lane] = __float2bfloat16_rn(du[j]);
                                }
                        }
                    } else if (rv == 32) {
                        stage_transposed_and_store(v, &map_o0, feat0, r0);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)   // rows past the tile belong to the expert's next tile, or to nobody
                            if (j < rv) p.out0[(long long)(r0 + j) * p.ldo + feat0 + lane] = __float2bfloat16_rn(v[j]);
                    }
                }
            } else if (swiglu(KIND)) {
                const int ng = tl.n0 >> 1;
                // full tile: gate in tensor-memory columns 0..127, up in 128..255, this warp takes two 32-column blocks.
                // half tile: this lane group's 64 features: gate in columns 0..63, up in 64..127, one block per warp.
                const int c_begin = half_tile ? half : 2 * half, c_end = half_tile ? half + 1 : 2 * half + 2;
                const int u_off = half_tile ? 64 : 128;
                const int x_base = ng + (half_tile ? (quarter >> 1) * 64 : 0);
#pragma unroll 1
                for (int c = c_begin; c < c_end; ++c) {
                    uint32_t g[32], u[32];
                    tc_ld32(taddr + c * 32, g);
                    tc_ld32(taddr + u_off + c * 32, u);
                    tc_wait_ld();
                    if (rows_valid == 0 || x_base + c * 32 >= p.I) continue;   // past the expert's rows / past column I
                    uint32_t hp[16], gp[16], up[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
                        const float u0 = __uint_as_float(u[2 * j]), u1 = __uint_as_float(u[2 * j + 1]);
                        const float h0 = __fdividef(g0, 1.f + __expf(-g0)) * u0;
                        const float h1 = __fdividef(g1, 1.f + __expf(-g1)) * u1;
                        hp[j] = pack_bf16(h0, h1);
                        gp[j] = pack_bf16(g0, g1);
                        up[j] = pack_bf16(u0, u1);
                    }
                    const int x = x_base + c * 32;
                    if (rows_valid == 32) {
                        stage_and_store(hp, &map_o0, x, slab_y);
                        if (p.gu) {
                            stage_and_store(gp, &map_o1, x, slab_y);
                            stage_and_store(up, &map_o1, p.I + x, slab_y);
                        }
                    } else if (lane < rows_valid) {
                        direct_store(hp, p.out0 + row * p.I + x);
                        if (p.gu) {
                            direct_store(gp, p.gu + row * (2ll * p.I) + x);
                            direct_store(up, p.gu + row * (2ll * p.I) + p.I + x);
                        }
                    }
                }
            } else {
                const bool have_acc = tl.k_blocks > 0;
                if (!have_acc && rows_valid == 32) {
                    zero_blocks(tl.n0 + half * (BN / 2), slab_y);
                } else if (fused_sb(KIND)) {
                    // row-major tile with the SwiGLU backward fused: per 32-column block, the accumulator (dHact, fp32)
                    // meets this row's g and u values (16-byte pieces of the lane's row of the two input blocks)
                    constexpr int NC = BN / 64;
                    const int c0 = half * NC;
                    int n_owed = 0;                      // blocks of this warp inside the I columns
                    for (int c = c0; c < c0 + NC; ++c) n_owed += (rows_valid != 0 && tl.n0 + c * 32 < p.n_cols) ? 1 : 0;
                    if (n_owed != 0) fetch_gu(tl.n0 + c0 * 32, slab0);
#pragma unroll 1
                    for (int i = 0; i < NC; ++i) {
                        uint32_t vr[32];
                        tc_ld32(taddr + (c0 + i) * 32, vr);
                        tc_wait_ld();
                        if (i >= n_owed) continue;
                        const int x = tl.n0 + (c0 + i) * 32;
                        if (!mbar_wait(gu_bar, gu_phase, abort_flag)) break;
                        gu_phase ^= 1u;
                        uint4 gq[4], uq[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            gq[j] = *reinterpret_cast<const uint4*>(g_blk + lane * 64 + ((j ^ sw) << 4));
                            uq[j] = *reinterpret_cast<const uint4*>(u_blk + lane * 64 + ((j ^ sw) << 4));
                        }
                        if (i + 1 < n_owed) {
                            // the next fetch overwrites the two input blocks: every lane's reads must have RETURNED
                            // (not merely been issued) before it starts
                            uint32_t seen = 0;
#pragma unroll
                            for (int j = 0; j < 4; ++j) seen ^= gq[j].x ^ gq[j].y ^ gq[j].z ^ gq[j].w ^ uq[j].x ^ uq[j].y ^ uq[j].z ^ uq[j].w;
                            inputs_consumed(seen);
                            fetch_gu(x + 32, slab0);
                        }
                        uint32_t dgp[16], dup[16];
                        const uint32_t* gw = reinterpret_cast<const uint32_t*>(gq);
                        const uint32_t* uw = reinterpret_cast<const uint32_t*>(uq);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float2 g2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[j]));
                            const float2 u2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&uw[j]));
                            float dg0, du0, dg1, du1;
                            swiglu_grad(__uint_as_float(vr[2 * j]), g2.x, u2.x, dg0, du0);
                            swiglu_grad(__uint_as_float(vr[2 * j + 1]), g2.y, u2.y, dg1, du1);
                            dgp[j] = pack_bf16(dg0, dg1);
                            dup[j] = pack_bf16(du0, du1);
                        }
                        if (rows_valid == 32) {
                            stage_and_store(dgp, &map_o0, x, slab_y);
                            stage_and_store(dup, &map_o0, p.I + x, slab_y);
                        } else if (lane < rows_valid) {
                            direct_store(dgp, p.out0 + row * p.ldo + x);
                            direct_store(dup, p.out0 + row * p.ldo + p.I + x);
                        }
                    }
                } else {
                    drain_plain(taddr, tl.n0, have_acc, rows_valid, slab_y, row);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR && rank != 0)
                    mbar_arrive_remote(acc == 0 ? tmem_empty_remote0 : tmem_empty_remote1);
                else
                    mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        // the staging buffer must have been read, and the stores completed, before the CTA exits
        if (n_stores != 0 && lane == 0) bulk_wait_all0();
        __syncwarp();
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // neither CTA's shared memory / barriers may go away while the other still uses them
    if (warp == 1) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                         : "memory");
    }
}

static_assert(Geo<false>::SMEM_BYTES <= 232448 && Geo<true>::SMEM_BYTES <= 232448 && Geo<true, true>::SMEM_BYTES <= 232448,
              "exceeds the 227 KB of shared memory a CTA can opt in to");

// ---- host side ------------------------------------------------------------------------------------
// MN-major operand [rows, cols] (cols contiguous) seen as {64 columns, rows, cols/64 chunks}: one box of
// {64, BK rows, n_chunks} lands chunk-major in shared memory, i.e. as n_chunks consecutive 64 x BK swizzled
// blocks -- the layout the MN-major UMMA descriptors expect.
bool make_map_mn(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint32_t n_chunks) {
    PFN_cuTensorMapEncodeTiled_v12000 fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {64, rows, cols / 64};
    cuuint64_t strides[2] = {cols * 2, 128};
    cuuint32_t box[3] = {64, (cuuint32_t)BK, n_chunks};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Grid of a launch: one CTA per SM (single), or as many CTA pairs as can be resident at once (pair).
// A pair that could not be co-scheduled would run after the others and double the kernel's duration,
// so the pair grid is sized from the occupancy query, per device and kernel.
// Swapped kinds: `a`, `o1` and `x` are the row operand's maps with boxes of 4, 2 and 1 times the smallest box
// (32 rows in pair mode, 64 otherwise); the other kinds pass `a` for `x`.
template <int KIND, bool PAIR>
int launch(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const CUtensorMap& o0,
           const CUtensorMap& o1, const CUtensorMap& x, const Params& p, cudaStream_t s) {
    static int grid_of_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOE_ERR_CUDA;
    auto kernel = grouped_gemm_kernel<KIND, PAIR>;
    if (grid_of_device[dev] == 0) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<PAIR, fused_sb(KIND)>::SMEM_BYTES) != cudaSuccess)
            return MOE_ERR_CUDA;
        const int sms = sm_count();
        if (sms <= 0) return MOE_ERR_CUDA;
        if (PAIR) {
            cudaLaunchConfig_t qc = {};
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
            qc.gridDim = dim3(2 * (sms / 2)); qc.blockDim = dim3(NUM_THREADS); qc.dynamicSmemBytes = Geo<PAIR, fused_sb(KIND)>::SMEM_BYTES;
            qc.attrs = qa; qc.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &qc) != cudaSuccess || clusters <= 0) return MOE_ERR_CUDA;
            if (clusters > sms / 2) clusters = sms / 2;
            grid_of_device[dev] = 2 * clusters;
        } else {
            grid_of_device[dev] = sms;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(grid_of_device[dev]);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = Geo<PAIR, fused_sb(KIND)>::SMEM_BYTES;
    cfg.stream = s;
    if (PAIR) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
    if (cudaLaunchKernelEx(&cfg, kernel, a, b0, b1, o0, o1, x, p) != cudaSuccess) return MOE_ERR_CUDA;
    return check_launch();
}

// The plain row-ragged GEMMs (down forward, down dgrad, gate/up dgrad) run with swapped operand roles -- always as
// CTA pairs: 256 output features x up to 256 rows per tile -- when experts hold fewer than 512 rows on average:
// there the fixed 128-row tiles lose 10-15 % of the tensor work to padding (measured: +2-5 % per kernel on the
// 384- and 451-rows-per-expert workloads).  With larger experts the padding is small and the fixed-height tiles
// are as fast or faster (the swapped kernels' issue thread, not the tensor pipe, bounds tiles of fewer than 256 rows).
bool use_swapped(const moe_dims_t& d) { return (long long)d.T * d.K < 512ll * d.E; }
// The SwiGLU forward has no swapped form (measured slower: two accumulators per tile).  Its pair kernel runs an
// expert's last <= 128 rows as a half-height tile, which makes pairs worthwhile from 320 rows per expert on average.
constexpr long long kSwigluPairRows = 320;
bool use_pairs_for_swiglu(const moe_dims_t& d) { return (long long)d.T * d.K >= kSwigluPairRows * d.E; }
// Weight gradients have no row padding to lose, so pairs already win from 256 rows per expert.
bool use_pairs_for_wgrad(const moe_dims_t& d) { return (long long)d.T * d.K >= 256ll * d.E; }

}  // namespace

// Gate/up forward: A = x_perm [R,H]; B = w_gate, w_up viewed as [E*H, I]; fused width 2I in tiles of
// 128 gate + 128 up columns.
int launch_gateup_fwd(const moe_dims_t& d, const bf16* x_perm, const bf16* w_gate, const bf16* w_up,
                      const int32_t* offsets, bf16* h_act, bf16* gu, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    const bool pair = use_pairs_for_swiglu(d);
    // pair mode with small experts (fewer than 512 rows on average): an expert's last <= 128 rows run as a half-height
    // tile; that takes one-chunk weight boxes (a half-height tile mixes gate and up chunks per CTA) and a second A map
    // with a 64-row box.  With larger experts the padding is small and the two-chunk boxes (one load less per stage)
    // are 2-4 % faster.
    const bool half_tiles = pair && use_swapped(d);
    CUtensorMap a, ah, b0, b1, o0, o1;
    if (!make_map(&a, x_perm, d.H, R, BK, BM) || !make_map(&ah, x_perm, d.H, R, BK, BM / 2) ||
        !make_map_mn(&b0, w_gate, d.I, (uint64_t)d.E * d.H, half_tiles ? 1 : 2) ||
        !make_map_mn(&b1, w_up, d.I, (uint64_t)d.E * d.H, half_tiles ? 1 : 2) || !make_out_map(&o0, h_act, d.I, R) ||
        !make_out_map(&o1, gu ? gu : h_act, gu ? 2ull * d.I : d.I, R))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.k_blocks = d.H / BK; p.k_split = p.k_blocks;
    p.n_tiles = (d.I + 127) / 128; p.n_cols = 2 * d.I; p.b_rows_per_e = d.H;
    p.out0 = h_act; p.gu = gu; p.I = d.I; p.ldo = d.I; p.n_split = 2 * d.I;
    if (half_tiles) return launch<FWD_SWIGLU_H, true>(a, b0, b1, o0, o1, ah, p, s);
    return pair ? launch<FWD_SWIGLU, true>(a, b0, b1, o0, o1, a, p, s) : launch<FWD_SWIGLU, false>(a, b0, b1, o0, o1, a, p, s);
}

// Down forward: A = h_act [R,I]; B = w_down viewed as [E*I, H].
int launch_down_fwd(const moe_dims_t& d, const bf16* h_act, const bf16* w_down, const int32_t* offsets,
                    bf16* y_perm, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    if (use_swapped(d)) {
        // swapped roles: M side = w_down tile (128 features of H, MN-major), N side = rows of h_act (64-row boxes)
        const int feats = 2 * SWAP_FEATS;   // a CTA pair's tile
        const uint32_t box = 32;            // row boxes of 32 / 64 / 128 rows per CTA
        CUtensorMap a, a2, a1, b0, o0;
        if (!make_map(&a, h_act, d.I, R, BK, 4 * box) || !make_map(&a2, h_act, d.I, R, BK, 2 * box) ||
            !make_map(&a1, h_act, d.I, R, BK, box) ||
            !make_map_mn(&b0, w_down, d.H, (uint64_t)d.E * d.I, SWAP_FEATS / 64) || !make_out_map(&o0, y_perm, d.H, R))
            return MOE_ERR_CUDA;
        Params p = {};
        p.offsets = offsets; p.E = d.E; p.k_blocks = d.I / BK; p.k_split = p.k_blocks;
        p.n_tiles = (d.H + feats - 1) / feats; p.n_cols = d.H; p.b_rows_per_e = d.I;
        p.out0 = y_perm; p.ldo = d.H; p.n_split = d.H;
        return launch<FWD_PLAIN_T, true>(a, b0, b0, o0, a2, a1, p, s);
    }
    // larger experts: 256-row pair tiles (each CTA loads half of B's columns)
    CUtensorMap a, b0, o0;
    if (!make_map(&a, h_act, d.I, R, BK, BM) || !make_map_mn(&b0, w_down, d.H, (uint64_t)d.E * d.I, BN / 128) ||
        !make_out_map(&o0, y_perm, d.H, R))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.k_blocks = d.I / BK; p.k_split = p.k_blocks;
    p.n_tiles = (d.H + BN - 1) / BN; p.n_cols = d.H; p.b_rows_per_e = d.I;
    p.out0 = y_perm; p.ldo = d.H; p.n_split = d.H;
    return launch<FWD_PLAIN, true>(a, b0, b0, o0, o0, a, p, s);
}

// Down dgrad: dh_act = dy_perm . w_down[e]^T.  A = dy_perm [R,H]; B = w_down viewed as [E*I, H] (rows are
// output columns, K = H contiguous).
int launch_down_dgrad(const moe_dims_t& d, const bf16* dy_perm, const bf16* w_down, const int32_t* offsets,
                      bf16* dh_act, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    if (use_swapped(d)) {
        // swapped roles: M side = w_down tile (128 features of I, K-major), N side = rows of dy_perm
        const int feats = 2 * SWAP_FEATS;   // a CTA pair's tile
        const uint32_t box = 32;            // row boxes of 32 / 64 / 128 rows per CTA
        CUtensorMap a, a2, a1, b0, o0;
        if (!make_map(&a, dy_perm, d.H, R, BK, 4 * box) || !make_map(&a2, dy_perm, d.H, R, BK, 2 * box) ||
            !make_map(&a1, dy_perm, d.H, R, BK, box) ||
            !make_map(&b0, w_down, d.H, (uint64_t)d.E * d.I, BK, SWAP_FEATS) || !make_out_map(&o0, dh_act, d.I, R))
            return MOE_ERR_CUDA;
        Params p = {};
        p.offsets = offsets; p.E = d.E; p.k_blocks = d.H / BK; p.k_split = p.k_blocks;
        p.n_tiles = (d.I + feats - 1) / feats; p.n_cols = d.I; p.b_rows_per_e = d.I;
        p.out0 = dh_act; p.ldo = d.I; p.n_split = d.I;
        return launch<DGRAD_T, true>(a, b0, b0, o0, a2, a1, p, s);
    }
    CUtensorMap a, b0, o0;
    if (!make_map(&a, dy_perm, d.H, R, BK, BM) || !make_map(&b0, w_down, d.H, (uint64_t)d.E * d.I, BK, BN / 2) ||
        !make_out_map(&o0, dh_act, d.I, R))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.k_blocks = d.H / BK; p.k_split = p.k_blocks;
    p.n_tiles = (d.I + BN - 1) / BN; p.n_cols = d.I; p.b_rows_per_e = d.I;
    p.out0 = dh_act; p.ldo = d.I; p.n_split = d.I;
    return launch<DGRAD, true>(a, b0, b0, o0, o0, a, p, s);
}

// Down dgrad with the SwiGLU backward in its epilogue: dgu = [dg | du] from dh = dy_perm . w_down[e]^T (kept in fp32)
// and the saved pre-activations gu [R, 2I].  Same operands and tile schedules as launch_down_dgrad; the epilogue
// warps fetch the [g | u] blocks through `g` (32 x 32 boxes of gu) and write two blocks of dgu per accumulator block.
int launch_down_dgrad_swiglu_bwd(const moe_dims_t& d, const bf16* dy_perm, const bf16* w_down, const bf16* gu,
                                 const int32_t* offsets, bf16* dgu, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    CUtensorMap g, o0;
    if (!make_out_map(&g, gu, 2ull * d.I, R) || !make_out_map(&o0, dgu, 2ull * d.I, R)) return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.k_blocks = d.H / BK; p.k_split = p.k_blocks;
    p.n_cols = d.I; p.b_rows_per_e = d.I; p.out0 = dgu; p.ldo = 2ll * d.I; p.n_split = d.I; p.I = d.I;
    if (use_swapped(d)) {
        const int feats = 2 * SWAP_FEATS;   // a CTA pair's tile
        const uint32_t box = 32;            // row boxes of 32 / 64 / 128 rows per CTA
        CUtensorMap a, a2, a1, b0;
        if (!make_map(&a, dy_perm, d.H, R, BK, 4 * box) || !make_map(&a2, dy_perm, d.H, R, BK, 2 * box) ||
            !make_map(&a1, dy_perm, d.H, R, BK, box) || !make_map(&b0, w_down, d.H, (uint64_t)d.E * d.I, BK, SWAP_FEATS))
            return MOE_ERR_CUDA;
        p.n_tiles = (d.I + feats - 1) / feats;
        return launch<DGRAD_T_SB, true>(a, b0, g, o0, a2, a1, p, s);
    }
    CUtensorMap a, b0;
    if (!make_map(&a, dy_perm, d.H, R, BK, BM) || !make_map(&b0, w_down, d.H, (uint64_t)d.E * d.I, BK, BN / 2))
        return MOE_ERR_CUDA;
    p.n_tiles = (d.I + BN - 1) / BN;
    return launch<DGRAD_SB, true>(a, b0, g, o0, o0, a, p, s);
}

// Gate/up dgrad: dx_perm = dg . w_gate[e]^T + du . w_up[e]^T.  A = dgu [R,2I]; the contraction runs over the
// gate half against w_gate viewed as [E*H, I], then over the up half against w_up.
int launch_gateup_dgrad(const moe_dims_t& d, const bf16* dgu, const bf16* w_gate, const bf16* w_up,
                        const int32_t* offsets, bf16* dx_perm, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    if (use_swapped(d)) {
        const int feats = 2 * SWAP_FEATS;   // a CTA pair's tile
        const uint32_t box = 32;            // row boxes of 32 / 64 / 128 rows per CTA
        CUtensorMap a, a2, a1, b0, b1, o0;
        if (!make_map(&a, dgu, 2ull * d.I, R, BK, 4 * box) || !make_map(&a2, dgu, 2ull * d.I, R, BK, 2 * box) ||
            !make_map(&a1, dgu, 2ull * d.I, R, BK, box) ||
            !make_map(&b0, w_gate, d.I, (uint64_t)d.E * d.H, BK, SWAP_FEATS) ||
            !make_map(&b1, w_up, d.I, (uint64_t)d.E * d.H, BK, SWAP_FEATS) || !make_out_map(&o0, dx_perm, d.H, R))
            return MOE_ERR_CUDA;
        Params p = {};
        p.offsets = offsets; p.E = d.E; p.k_blocks = 2 * d.I / BK; p.k_split = d.I / BK;
        p.n_tiles = (d.H + feats - 1) / feats; p.n_cols = d.H; p.b_rows_per_e = d.H;
        p.out0 = dx_perm; p.ldo = d.H; p.n_split = d.H;
        return launch<DGRAD_T, true>(a, b0, b1, o0, a2, a1, p, s);
    }
    const uint32_t bn = BN / 2;
    CUtensorMap a, b0, b1, o0;
    if (!make_map(&a, dgu, 2ull * d.I, R, BK, BM) || !make_map(&b0, w_gate, d.I, (uint64_t)d.E * d.H, BK, bn) ||
        !make_map(&b1, w_up, d.I, (uint64_t)d.E * d.H, BK, bn) || !make_out_map(&o0, dx_perm, d.H, R))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.k_blocks = 2 * d.I / BK; p.k_split = d.I / BK;
    p.n_tiles = (d.H + BN - 1) / BN; p.n_cols = d.H; p.b_rows_per_e = d.H;
    p.out0 = dx_perm; p.ldo = d.H; p.n_split = d.H;
    return launch<DGRAD, true>(a, b0, b1, o0, o0, a, p, s);
}

// Weight gradients: the tile grid is static (M x N per expert).  Pairs (256 x 256 tiles) pay off once an
// expert's contraction is long enough to amortise the pair's per-tile hand-shakes; with few rows per expert
// the independent 128 x 256 tiles are faster.
// Down wgrad: dw_down[e] [I,H] = h_act_e^T . dy_perm_e.  A = h_act [R,I] (M = I), B = dy_perm [R,H] (N = H).
int launch_down_wgrad(const moe_dims_t& d, const bf16* h_act, const bf16* dy_perm, const int32_t* offsets,
                      bf16* dw_down, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    const bool pair = use_pairs_for_wgrad(d);
    const int tile_m = pair ? 2 * BM : BM;
    CUtensorMap a, b0, o0;
    if (!make_map_mn(&a, h_act, d.I, R, BM / 64) || !make_map_mn(&b0, dy_perm, d.H, R, pair ? BN / 128 : BN / 64) ||
        !make_out_map(&o0, dw_down, d.H, (uint64_t)d.E * d.I))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.m_rows = d.I; p.m_tiles = (d.I + tile_m - 1) / tile_m;
    p.n_tiles = (d.H + BN - 1) / BN; p.n_cols = d.H; p.n_split = d.H; p.ldo = d.H;
    p.out0 = dw_down; p.out1 = nullptr;
    return pair ? launch<WGRAD, true>(a, b0, b0, o0, o0, a, p, s) : launch<WGRAD, false>(a, b0, b0, o0, o0, a, p, s);
}

// Gate/up wgrad (the paper's dW1): [dw_gate[e] | dw_up[e]] = x_perm_e^T . dgu_e.  A = x_perm [R,H] (M = H),
// B = dgu [R,2I] (N = 2I); output columns below I go to dw_gate, the rest to dw_up.
int launch_gateup_wgrad(const moe_dims_t& d, const bf16* x_perm, const bf16* dgu, const int32_t* offsets,
                        bf16* dw_gate, bf16* dw_up, cudaStream_t s) {
    const uint64_t R = (uint64_t)d.T * d.K;
    const bool pair = use_pairs_for_wgrad(d);
    const int tile_m = pair ? 2 * BM : BM;
    CUtensorMap a, b0, o0, o1;
    if (!make_map_mn(&a, x_perm, d.H, R, BM / 64) || !make_map_mn(&b0, dgu, 2ull * d.I, R, pair ? BN / 128 : BN / 64) ||
        !make_out_map(&o0, dw_gate, d.I, (uint64_t)d.E * d.H) || !make_out_map(&o1, dw_up, d.I, (uint64_t)d.E * d.H))
        return MOE_ERR_CUDA;
    Params p = {};
    p.offsets = offsets; p.E = d.E; p.m_rows = d.H; p.m_tiles = (d.H + tile_m - 1) / tile_m;
    p.n_tiles = (2 * d.I + BN - 1) / BN; p.n_cols = 2 * d.I; p.n_split = d.I; p.ldo = d.I;
    p.out0 = dw_gate; p.out1 = dw_up;
    return pair ? launch<WGRAD, true>(a, b0, b0, o0, o1, a, p, s) : launch<WGRAD, false>(a, b0, b0, o0, o1, a, p, s);
}

}  // namespace moe
