// Device code of the fused vocabulary projection + cross-entropy: kernel parameters, the four
// epilogues (fold, residual, input gradient, weight gradient), the single-CTA and the CTA-pair GEMM
// kernels, and the small merge / count / mean kernels.  See vp_ce.cu for the overall description.
#pragma once

#include "sm100_ptx.cuh"
#include "vp_ce.h"

namespace vpce {


constexpr int BM = 128;          // accumulator rows per tile (TMEM lanes)
constexpr int BK = 64;           // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int UMMA_K = 16;       // K per tcgen05.mma for 16-bit inputs
constexpr int BN_VOCAB = 256;    // vocabulary columns per strip tile
constexpr int NUM_THREADS = 192;
constexpr int SMEM_BUDGET = 200 * 1024;    // operand stages
constexpr int SMEM_BUDGET_STAGED = 193 * 1024;   // operand stages of a kernel that also stages its output tile
constexpr int SMEM_EXTRA = 2048;           // barriers + alignment slack
// Output staging of every epilogue that writes a tile (all but the fold): per epilogue warp two 32-row x 128-byte
// boxes (64 bf16 or 32 fp32 columns) that leave through TMA stores / reductions.
constexpr int G_STAGING_BYTES = 4 * 2 * 4096;

enum Epilogue { EPI_FOLD = 0, EPI_RESID = 1, EPI_DH = 2, EPI_DW = 3 };

struct GemmParams {
    int m_tiles, n_tiles, num_kb;
    int a_3d, b_3d;                        // MN-major operand fetched as one 3-D box (64 x 64 x chunks) per k-block
    int hint_a, hint_b, hint_c;            // L2 eviction hints for A loads, B loads, C stores: 0 normal, 1 first, 2 last
    int n_cut, k_split, k_stagger;         // pair kernel, gradient GEMMs: the last n_cut tiles of the list run as k_split parts along K,
                                           // part j + 1 longer than part j by k_stagger k-blocks
    int* split_flags;                      // [n_cut][8] zero before the launch: order of the parts' additions (see the pair kernel)
    int group_n;                           // n-tiles per raster group (tiles run m-major inside a group)
    int a_mn0, a_k0, b_mn0, b_k0;          // TMA coordinate bases (elements)
    int rows_valid;                        // valid accumulator rows overall (M bound)
    int cols_valid;                        // valid accumulator columns overall (N bound)
    // FOLD / RESID
    int v_lo;                              // first vocabulary id of the shard
    const int32_t* labels;                 // chunk base
    const float* lse;                      // chunk base
    const float* dloss;                    // chunk base or null
    const float* inv_n_valid;              // scalar used when dloss == null
    int ignore_index;
    int V;
    float* pm;                             // [n_tile][part_ld] partial max
    float* pz;                             // [n_tile][part_ld] partial sum-exp
    float* ylab;                           // [part_ld] target logit
    int part_ld;
    __nv_bfloat16* G;                      // [T_chunk][g_ld]
    float* delta;                          // [T_chunk] or null: exact minus bf16-rounded value of each token's target entry of G
    int g_ld;
    int g_rows;                            // rows of the G workspace (T_chunk)
    // DH / DW: the fp32 output is described by the launch's third tensor map (boxes of 32 columns x 32 rows)
    int c_row0;                            // output row of accumulator row 0 of tile 0 (map coordinates)
    int accumulate;                        // 0: the tile is stored; else it is added to the output (TMA reduction)
    int* status;
    int* tile_counter;                     // zero before the launch; tiles are taken with atomicAdd
    unsigned long long wait_limit_ns;      // every wait inside the kernel gives up after this long
    // Test hook (host-side injection of a lost signal; nothing is accessed out of bounds): the CTA (pair) that takes
    // list position 0 does not issue the copies of k-block drop_kb of that tile, so the stage's "full" barrier never
    // completes and the waits run out.  drop_kb < 0: off.  drop_ranks: bit r set = CTA rank r of the pair drops
    // (bit 0 alone for the single-CTA kernel).
    int drop_kb, drop_ranks;
};

template <int BN, int EPI = EPI_FOLD> struct StageCfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int BUDGET = EPI == EPI_FOLD ? SMEM_BUDGET : SMEM_BUDGET_STAGED;
    static constexpr int STAGES = (BUDGET / STAGE_BYTES) > 8 ? 8 : (BUDGET / STAGE_BYTES);
    // every epilogue but the fold stages its output tile in shared memory for TMA stores
    static constexpr int SMEM_TOTAL = STAGES * STAGE_BYTES + SMEM_EXTRA + (EPI == EPI_FOLD ? 0 : G_STAGING_BYTES);
    static_assert(SMEM_TOTAL <= 227 * 1024, "shared memory per CTA");
};
template <int BN, int EPI> constexpr int smem_total() { return StageCfg<BN, EPI>::SMEM_TOTAL; }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

// Tile order: the n-tiles are cut into groups of group_n; inside a group the index runs n-fastest
// over all m-tiles, so the group's B operand (a slice of the shard) stays in L2 while A streams.
__device__ __forceinline__ void decode_tile(const GemmParams& p, int tile, int& mt, int& nt) {
    const int per_group = p.group_n * p.m_tiles;
    const int g = tile / per_group;
    const int r = tile - g * per_group;
    const int n0 = g * p.group_n;
    const int gw = min(p.group_n, p.n_tiles - n0);
    mt = r / gw;
    nt = n0 + (r - mt * gw);
}

// ------------------------------------------------------------------------------------ epilogues
// Each epilogue thread owns accumulator row `row` (0..127) of the tile; `tmem_row` is the
// TMEM address of that thread's lane quadrant at the accumulator's first column.
constexpr float LOG2E = 1.4426950408889634f;
constexpr float NEG_INF = -__builtin_huge_valf();

__device__ __forceinline__ void epilogue_fold(const GemmParams& p, int mt, int nt, int row, uint32_t tmem_row) {
    const int grow = mt * BM + row;                             // row within the chunk
    const bool row_ok = grow < p.rows_valid;
    const int label = row_ok ? p.labels[grow] : -1;
    // target column relative to the tile; a target beyond the shard's last valid column belongs to another shard
    // (its padded column here holds no logit)
    const int lrel = (label - p.v_lo < p.cols_valid) ? label - (p.v_lo + nt * BN_VOCAB) : -1;
    float m = NEG_INF, z = 0.f, yl = 0.f;
    bool hit = false;
#pragma unroll 1
    for (int c = 0; c < BN_VOCAB / 32; ++c) {
        float v[32];
        __syncwarp();
        tmem_ld32(tmem_row + c * 32, v);
        tmem_ld_wait();
        const int nvalid = p.cols_valid - (nt * BN_VOCAB + c * 32);     // valid columns left in the shard
        if (nvalid < 32) {
#pragma unroll
            for (int j = 0; j < 32; ++j) if (j >= nvalid) v[j] = NEG_INF;
        }
        if (static_cast<unsigned>(lrel - c * 32) < 32u) {
            const int jj = lrel - c * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) if (j == jj) yl = v[j];
            hit = true;
        }
        float cmax = v[0];
#pragma unroll
        for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, v[j]);
        const float m_new = fmaxf(m, cmax);
        const float mL = (m_new == NEG_INF) ? 0.f : m_new * LOG2E;
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) s += ex2f(fmaf(v[j], LOG2E, -mL));
        z = z * ex2f(fmaf(m, LOG2E, -mL)) + s;                         // m = -inf gives factor 0
        m = m_new;
    }
    if (row_ok) {
        p.pm[static_cast<size_t>(nt) * p.part_ld + grow] = m;
        p.pz[static_cast<size_t>(nt) * p.part_ld + grow] = z;
        if (hit) p.ylab[grow] = yl;                                    // exactly one tile owns the target
    }
}

// The bf16 residual tile leaves through shared memory: each epilogue warp owns 32 rows; per 64
// columns it fills a 32 x 128-byte box (128-byte swizzle: 16-byte chunk j of row r sits at chunk
// j ^ (r & 7)) and one lane issues a TMA store, so global writes are whole 128-byte lines.
__device__ __forceinline__ void epilogue_resid(const GemmParams& p, const CUtensorMap* tmG, uint32_t stage_smem,
                                               int mt, int nt, int row, int lane, uint32_t tmem_row) {
    const int grow = mt * BM + row;
    const bool row_ok = grow < p.rows_valid;
    int label = row_ok ? p.labels[grow] : p.ignore_index;
    const bool valid = row_ok && label != p.ignore_index && static_cast<unsigned>(label) < static_cast<unsigned>(p.V);
    // a label outside [0, V) is treated as ignored and flagged (once per row: by the strip's first tile)
    if (row_ok && !valid && label != p.ignore_index && nt == 0) atomicOr(p.status, VPCE_DEV_LABEL_OUT_OF_RANGE);
    float dl = 0.f, lseL = 0.f;
    if (valid) dl = p.dloss ? p.dloss[grow] : *p.inv_n_valid;
    if (row_ok) lseL = p.lse[grow] * LOG2E;
    const int lrel = valid ? label - (p.v_lo + nt * BN_VOCAB) : -1;
    const uint64_t pol_c = make_policy(p.hint_c);
#pragma unroll 1
    for (int h = 0; h < BN_VOCAB / 64; ++h) {
        const uint32_t buf = stage_smem + (h & 1) * 4096;
        if (lane == 0) bulk_wait_read_1();                              // the store that last read this buffer is done
        __syncwarp();
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
            const int c = 2 * h + c2;
            float v[32];
            __syncwarp();
            tmem_ld32(tmem_row + c * 32, v);
            tmem_ld_wait();
            const int nvalid = p.cols_valid - (nt * BN_VOCAB + c * 32);
            const int jj = lrel - c * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                float g = dl * ex2f(fmaf(v[j], LOG2E, -lseL));
                if (j == jj) g -= dl;
                v[j] = (j < nvalid) ? g : 0.f;
            }
            if (static_cast<unsigned>(jj) < 32u && jj < nvalid && p.delta) {
                // what bf16 rounding takes from this token's one-hot entry; the fix-up kernels add it back exactly
                float gx = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) if (j == jj) gx = v[j];
                p.delta[grow] = gx - __bfloat162float(__float2bfloat16_rn(gx));
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint4 o;
                o.x = pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
                o.y = pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
                o.z = pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
                o.w = pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
                const int chunk = c2 * 4 + q;                           // 16-byte chunk within the 128-byte row
                st_shared_v4(buf + lane * 128 + ((chunk ^ (lane & 7)) << 4), o);   // rows >= rows_valid get zeros
            }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0 && mt * BM < p.g_rows) {                          // tiles past the workspace rows store nothing
            if (p.hint_c) tma_store_2d_hint(tmG, buf, nt * BN_VOCAB + h * 64, mt * BM + (row - lane), pol_c);
            else tma_store_2d(tmG, buf, nt * BN_VOCAB + h * 64, mt * BM + (row - lane));
            bulk_commit();
        }
    }
}

// fp32 variant for the TF32 path: per 32 columns a 32 x 128-byte box of floats.
__device__ __forceinline__ void epilogue_resid_f32(const GemmParams& p, const CUtensorMap* tmG, uint32_t stage_smem,
                                                   int mt, int nt, int row, int lane, uint32_t tmem_row) {
    const int grow = mt * BM + row;
    const bool row_ok = grow < p.rows_valid;
    int label = row_ok ? p.labels[grow] : p.ignore_index;
    const bool valid = row_ok && label != p.ignore_index && static_cast<unsigned>(label) < static_cast<unsigned>(p.V);
    // a label outside [0, V) is treated as ignored and flagged (once per row: by the strip's first tile)
    if (row_ok && !valid && label != p.ignore_index && nt == 0) atomicOr(p.status, VPCE_DEV_LABEL_OUT_OF_RANGE);
    float dl = 0.f, lseL = 0.f;
    if (valid) dl = p.dloss ? p.dloss[grow] : *p.inv_n_valid;
    if (row_ok) lseL = p.lse[grow] * LOG2E;
    const int lrel = valid ? label - (p.v_lo + nt * BN_VOCAB) : -1;
    const uint64_t pol_c = make_policy(p.hint_c);
#pragma unroll 1
    for (int c = 0; c < BN_VOCAB / 32; ++c) {
        const uint32_t buf = stage_smem + (c & 1) * 4096;
        if (lane == 0) bulk_wait_read_1();
        __syncwarp();
        float v[32];
        tmem_ld32(tmem_row + c * 32, v);
        tmem_ld_wait();
        const int nvalid = p.cols_valid - (nt * BN_VOCAB + c * 32);
        const int jj = lrel - c * 32;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            float g = dl * ex2f(fmaf(v[j], LOG2E, -lseL));
            if (j == jj) g -= dl;
            v[j] = (j < nvalid) ? g : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint4 o;
            o.x = __float_as_uint(v[4 * q]); o.y = __float_as_uint(v[4 * q + 1]);
            o.z = __float_as_uint(v[4 * q + 2]); o.w = __float_as_uint(v[4 * q + 3]);
            st_shared_v4(buf + lane * 128 + ((q ^ (lane & 7)) << 4), o);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0 && mt * BM < p.g_rows) {
            if (p.hint_c) tma_store_2d_hint(tmG, buf, nt * BN_VOCAB + c * 32, mt * BM + (row - lane), pol_c);
            else tma_store_2d(tmG, buf, nt * BN_VOCAB + c * 32, mt * BM + (row - lane));
            bulk_commit();
        }
    }
}

// fp32 output tile of the two gradient GEMMs.  Each epilogue warp owns 32 accumulator rows; per 32 columns it fills a
// 32 x 128-byte box in shared memory (128-byte swizzle: 16-byte chunk q of row r sits at chunk q ^ (r & 7)) and one
// lane hands it to the TMA unit, either as a store (the first contribution to this output) or as a reduction that ADDS
// the box to what global memory holds (fp32, done at the L2: the running sum never travels back to the SM).  Global
// traffic is whole 128-byte lines, and rows or columns outside the output's extent (the tensor map's) are dropped by
// the TMA unit, so no thread needs a bounds check.  Every output element receives exactly one contribution per launch
// and launches are ordered by the stream, so the sum's order is fixed.
// x0: first output column of the tile; y0: output row of this warp's first accumulator row; n_this: tile width.
__device__ __forceinline__ void epilogue_f32_tile(const CUtensorMap* tmC, uint32_t stage_smem, int x0, int y0, int lane,
                                                  uint32_t tmem_row, int n_this, bool reduce) {
#pragma unroll 1
    for (int c = 0; c < (n_this + 31) / 32; ++c) {
        const uint32_t buf = stage_smem + (c & 1) * 4096;
        if (lane == 0) bulk_wait_read_1();                              // the copy that last read this buffer is done
        __syncwarp();
        float v[32];
        tmem_ld32(tmem_row + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint4 o;
            o.x = __float_as_uint(v[4 * q]); o.y = __float_as_uint(v[4 * q + 1]);
            o.z = __float_as_uint(v[4 * q + 2]); o.w = __float_as_uint(v[4 * q + 3]);
            st_shared_v4(buf + lane * 128 + ((q ^ (lane & 7)) << 4), o);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
            if (reduce) tma_reduce_add_2d(tmC, buf, x0 + c * 32, y0);
            else tma_store_2d(tmC, buf, x0 + c * 32, y0);
            bulk_commit();
        }
    }
}

// ------------------------------------------------------------------------------------ the GEMM kernel
// Tiles are handed out dynamically: the producer lane takes the next tile index from a global
// counter (atomicAdd) and publishes it to the MMA lane and the epilogue warps through a small
// shared-memory ring guarded by mbarriers, so a CTA that finishes early simply takes more tiles.
// The last n-tile of a row may be narrower than BN (its MMA uses N = valid columns rounded up
// to 16), so an output width that is not a multiple of BN costs no padded tensor-core work.
constexpr int SCHED_DEPTH = 8;

template <int BN, bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
vpce_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
    using Cfg = StageCfg<BN, EPI>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr uint32_t TMEM_COLS = (BN > 128) ? 512u : (BN > 64 ? 256u : 128u);
    constexpr uint32_t ACC_STRIDE = TMEM_COLS / 2;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                      // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t bars = base + STAGES * Cfg::STAGE_BYTES;            // 8-byte barriers after the stages
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
    const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);
    auto sfull_bar = [&](int s) { return bars + 8u * (2 * STAGES + 5 + s); };
    auto sempty_bar = [&](int s) { return bars + 8u * (2 * STAGES + 5 + SCHED_DEPTH + s); };
    constexpr int NUM_BARS = 2 * STAGES + 5 + 2 * SCHED_DEPTH;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + STAGES * Cfg::STAGE_BYTES + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* sched_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [SCHED_DEPTH] tile ids
    const uint32_t g_staging = base + STAGES * Cfg::STAGE_BYTES + 1024;   // RESID only (1024-byte aligned)

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        mbar_init(drain_bar, 1);
        for (int s = 0; s < SCHED_DEPTH; ++s) { mbar_init(sfull_bar(s), 1); mbar_init(sempty_bar(s), 5); }
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Valid accumulator columns of n-tile nt, rounded up to the MMA's granularity of 16.
    auto tile_n = [&](int nt) {
        const int left = p.cols_valid - nt * BN;
        return left >= BN ? BN : ((left + 15) & ~15);
    };

    if (warp == 0) {
        // ---------------------------------------------------------------- scheduler + TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            long issued = 0;
            const uint64_t pol_a = make_policy(p.hint_a), pol_b = make_policy(p.hint_b);
            const bool use_a = p.hint_a != 0, use_b = p.hint_b != 0;
            auto load_a = [&](uint32_t dst, uint32_t bar, int c0, int c1) {
                if (use_a) tma_load_2d_hint(dst, &tmA, bar, c0, c1, pol_a); else tma_load_2d(dst, &tmA, bar, c0, c1);
            };
            auto load_b = [&](uint32_t dst, uint32_t bar, int c0, int c1) {
                if (use_b) tma_load_2d_hint(dst, &tmB, bar, c0, c1, pol_b); else tma_load_2d(dst, &tmB, bar, c0, c1);
            };
            // The loads of one k-block of one tile into a stage.
            auto issue = [&](int mt, int nt, int kb, uint32_t sa, uint32_t sb, uint32_t bar) {
                if (A_MN && p.a_3d) {
                    const int c1 = p.a_k0 + kb * BK, c2 = (p.a_mn0 + mt * BM) >> 6;
                    if (use_a) tma_load_3d_hint(sa, &tmA, bar, 0, c1, c2, pol_a); else tma_load_3d(sa, &tmA, bar, 0, c1, c2);
                } else if (A_MN) {
#pragma unroll
                    for (int j = 0; j < BM / 64; ++j)
                        load_a(sa + j * (BK * 128), bar, p.a_mn0 + mt * BM + 64 * j, p.a_k0 + kb * BK);
                } else {
                    load_a(sa, bar, p.a_k0 + kb * BK, p.a_mn0 + mt * BM);
                }
                if (B_MN && p.b_3d) {
                    const int c1 = p.b_k0 + kb * BK, c2 = (p.b_mn0 + nt * BN) >> 6;
                    if (use_b) tma_load_3d_hint(sb, &tmB, bar, 0, c1, c2, pol_b); else tma_load_3d(sb, &tmB, bar, 0, c1, c2);
                } else if (B_MN) {
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j)
                        load_b(sb + j * (BK * 128), bar, p.b_mn0 + nt * BN + 64 * j, p.b_k0 + kb * BK);
                } else {
                    load_b(sb, bar, p.b_k0 + kb * BK, p.b_mn0 + nt * BN);
                }
            };
            while (ok) {
                if (!mbar_wait(sempty_bar(ss), sphase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                int tile = atomicAdd(p.tile_counter, 1);
                if (tile >= total_tiles) tile = -1;
                sched_slot[ss] = tile;
                mbar_arrive(sfull_bar(ss));                              // release: the slot is visible to waiters
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int mt, nt;
                decode_tile(p, tile, mt, nt);
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    mbar_arrive_expect_tx(full_bar(stage), Cfg::STAGE_BYTES);
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const bool drop = tile == 0 && kb == p.drop_kb && (p.drop_ranks & 1);   // test hook: a lost copy
                    if (!drop) issue(mt, nt, kb, sa, sa + Cfg::A_BYTES, full_bar(stage));
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok || *abort_flag) {
                // Give-up path: let this CTA's copies in flight land before shared memory is released.
                const long back = issued < STAGES ? issued : STAGES;
                int s = stage; uint32_t ph = phase;
                for (long i = 0; i < back; ++i) {
                    if (--s < 0) { s = STAGES - 1; ph ^= 1u; }
                    unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(s), ph) && globaltimer_ns() - t0 < p.wait_limit_ns) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            for (int it = 0; ok; ++it) {
                if (!mbar_wait(sfull_bar(ss), sphase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                const int tile = sched_slot[ss];
                mbar_arrive(sempty_bar(ss));
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int mt, nt;
                decode_tile(p, tile, mt, nt);
                const uint32_t idesc = make_idesc(tile_n(nt), A_MN, B_MN, BM);
                const int ab = it & 1;
                const uint32_t aphase = (it >> 1) & 1u;
                if (!mbar_wait(tempty_bar(ab), aphase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + ab * ACC_STRIDE;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    const uint64_t adesc = A_MN ? make_smem_desc(sa, BK * 128, 1024) : make_smem_desc(sa, 16, 1024);
                    const uint64_t bdesc = B_MN ? make_smem_desc(sb, BK * 128, 1024) : make_smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // K-major: 16 elements = 32 B along the swizzled row; MN-major: 16 K-rows = 2048 B
                        const uint64_t aoff = static_cast<uint64_t>((A_MN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        const uint64_t boff = static_cast<uint64_t>((B_MN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        umma_f16(tmem_d, adesc + aoff, bdesc + boff, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));                      // frees the stage once these MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(ab));
            }
            if (!ok || *abort_flag) {
                umma_commit(drain_bar);                                 // wait for MMAs still in flight
                unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(drain_bar, 0) && globaltimer_ns() - t0 < p.wait_limit_ns) {}
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int quad = warp & 3;                                     // TMEM lane quadrant this warp may read
        const int row = quad * 32 + lane;
        int ss = 0; uint32_t sphase = 0;
        bool ok = true;
        for (int it = 0; ok; ++it) {
            int tile = -2;
            if (lane == 0) {
                if (mbar_wait(sfull_bar(ss), sphase, abort_flag, p.wait_limit_ns)) {
                    tile = sched_slot[ss];
                    mbar_arrive(sempty_bar(ss));
                }
            }
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
            if (tile < 0) break;                                        // -1: no tiles left, -2: gave up
            int mt, nt;
            decode_tile(p, tile, mt, nt);
            const int ab = it & 1;
            const uint32_t aphase = (it >> 1) & 1u;
            if (!mbar_wait(tfull_bar(ab), aphase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tmem_row = tmem_base + ab * ACC_STRIDE + (static_cast<uint32_t>(quad * 32) << 16);
            if (EPI == EPI_FOLD) epilogue_fold(p, mt, nt, row, tmem_row);
            else if (EPI == EPI_RESID) epilogue_resid(p, &tmC, g_staging + (warp - 2) * 8192, mt, nt, row, lane, tmem_row);
            else epilogue_f32_tile(&tmC, g_staging + (warp - 2) * 8192, nt * BN, p.c_row0 + mt * BM + quad * 32, lane,
                                   tmem_row, tile_n(nt), p.accumulate != 0);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(ab));
        }
        if (EPI != EPI_FOLD && lane == 0) bulk_wait_all();              // staged stores / reductions have landed
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, VPCE_DEV_WAIT_EXPIRED);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------ the CTA-pair GEMM kernel
// Two CTAs of a cluster (one TPC) work on one 256 x BN tile with tcgen05.mma.cta_group::2: each
// CTA loads its own 128 rows of A and HALF of the B tile (BN/2 rows), the leader CTA (cluster rank
// 0) issues the MMAs, which read both CTAs' shared memory and write both CTAs' tensor memory, and
// each CTA drains its own 128 accumulator rows.  Per CTA and k-block this moves 16 KB + BN*64 B
// from L2 instead of 16 KB + BN*128 B: a third less L2->SM traffic at BN = 256.
// Signalling: TMA byte counts of both CTAs are credited to the leader's "full" barrier
// (.cta_group::2 loads, no multicast); tcgen05.commit with a CTA mask releases the stage in both
// CTAs and publishes the accumulator to both epilogues; epilogue warps of both CTAs arrive on the
// leader's "accumulator free" barrier.  Work is handed out dynamically: the leader takes list positions
// from the launch's counter and publishes them to both CTAs through a small ring (see below).
// With TF32 = true the operands are 32-bit floats multiplied as TF32 (kind::tf32, K = 8 per MMA,
// k-blocks of 32 elements); the 128-byte rows and hence all byte sizes are the same.
// The kernels that write an output tile give 32 KB of the 227 KB to its staging (6 stages); the fold kernel uses them
// for a 7th stage.
template <int BN, int EPI = EPI_RESID> struct PairCfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = (BN / 2) * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int BUDGET = SMEM_BUDGET + (EPI == EPI_FOLD ? 28 * 1024 : 0);
    static constexpr int STAGES = (BUDGET / STAGE_BYTES) > 8 ? 8 : (BUDGET / STAGE_BYTES);
    static constexpr int SMEM_TOTAL = STAGES * STAGE_BYTES + SMEM_EXTRA;
};
template <int BN, int EPI> constexpr int pair_smem_total() {
    return PairCfg<BN, EPI>::SMEM_TOTAL + (EPI == EPI_FOLD ? 0 : G_STAGING_BYTES);
}

template <int BN, bool A_MN, bool B_MN, int EPI, bool TF32 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
vpce_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
    using Cfg = PairCfg<BN, EPI>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr uint32_t TMEM_COLS = 512u;
    constexpr uint32_t ACC_STRIDE = 256u;
    static_assert(BN == 256, "pair tiles are 256 x 256");
    // Element-size dependent geometry: a 128-byte swizzled row holds BKE elements (one k-block of a K-major
    // operand, one chunk of an MN-major operand); one MMA consumes UK of them along K.
    constexpr int BKE = TF32 ? 32 : 64;
    constexpr int CSH = TF32 ? 5 : 6;
    constexpr int UK = TF32 ? 8 : 16;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t bars = base + STAGES * Cfg::STAGE_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };                    // used in the leader only
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };   // used in the leader only
    const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);
    auto sfull_bar = [&](int s) { return bars + 8u * (2 * STAGES + 5 + s); };
    auto sempty_bar = [&](int s) { return bars + 8u * (2 * STAGES + 5 + SCHED_DEPTH + s); };   // used in the leader only
    constexpr int NUM_BARS = 2 * STAGES + 5 + 2 * SCHED_DEPTH;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + STAGES * Cfg::STAGE_BYTES + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* sched_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [SCHED_DEPTH] list positions
    const uint32_t sched_slot_addr = bars + 8u * NUM_BARS + 8u;
    const uint32_t g_staging = base + STAGES * Cfg::STAGE_BYTES + 1024;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int pm_tiles = (p.m_tiles + 1) >> 1;                               // 256-row tiles

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
        mbar_init(drain_bar, 1);
        // a slot is free again when the leader's MMA lane + 4 epilogue warps and the peer's producer + 4 epilogue
        // warps have read it: 10 arrivals on the leader's barrier
        for (int s = 0; s < SCHED_DEPTH; ++s) { mbar_init(sfull_bar(s), 1); mbar_init(sempty_bar(s), 10); }
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem2_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem2_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                      // the peer's barriers exist before any remote signal
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // MMA width of n-tile nt.  Each CTA supplies N/2 columns of B: N/2 must be a multiple of 16, and
    // of 64 (one swizzled chunk) when B is MN-major.
    auto tile_n = [&](int nt) {
        const int left = p.cols_valid - nt * BN;
        constexpr int R = B_MN ? 2 * BKE : 32;
        return left >= BN ? BN : ((left + R - 1) / R * R);
    };
    // The work list, handed out dynamically (greedy list scheduling):
    //   [0, n_whole)                      256-row x BN tiles in raster order: n-fastest over ALL n-tiles of a row inside
    //                                     raster groups, so the narrower last n-tile of a row runs next to the row's other
    //                                     tiles and shares their A rows through L2;
    //   [n_whole, n_whole + ks * n_cut)   the last n_cut tiles as ks parts each along K (gradient GEMMs only; the host
    //                                     picks n_cut and ks so that the last round of the list ends sooner).  Part j + 1
    //                                     is k_stagger k-blocks longer than part j: parts taken together then finish one
    //                                     after the other, an epilogue apart, instead of queueing.  The parts of a tile add
    //                                     into the same output elements, in the order of j: each epilogue warp waits for
    //                                     the warp that wrote the same rows of part j - 1 (a flag in global memory), so the
    //                                     fp32 sum has one fixed order whatever pairs ran the parts.  A part is always taken
    //                                     from the list after the parts it waits for, and those never wait for a later
    //                                     entry, so the waits cannot form a cycle.
    constexpr bool kSplit = (EPI == EPI_DH || EPI == EPI_DW);
    const int total_tiles = pm_tiles * p.n_tiles;
    const int n_cut = kSplit ? min(p.n_cut, total_tiles) : 0;
    const int ks = n_cut > 0 ? max(p.k_split, 1) : 1;
    const int n_whole = total_tiles - n_cut;
    const int list_len = n_whole + ks * n_cut;
    auto decode_raster = [&](int tile, int& pmt, int& nt) {
        const int per_group = p.group_n * pm_tiles;
        const int g = tile / per_group;
        const int r = tile - g * per_group;
        const int n0 = g * p.group_n;
        const int gw = min(p.group_n, p.n_tiles - n0);
        pmt = r / gw;
        nt = n0 + (r - pmt * gw);
    };
    // Entry t of the list: 256-row tile pmt, n-tile nt (columns [ncol0, ncol0 + width)), k-blocks [kb0, kb1);
    // part j of split tile number `slot` (slot < 0: a whole tile).
    struct Work { int pmt, nt, ncol0, width, kb0, kb1, part, slot; };
    auto get_tile = [&](int t) {
        Work w;
        if (t < n_whole) {
            decode_raster(t, w.pmt, w.nt);
            w.kb0 = 0; w.kb1 = p.num_kb; w.part = 0; w.slot = -1;
        } else {
            const int v = t - n_whole;
            w.slot = v / ks;
            w.part = v - w.slot * ks;
            decode_raster(n_whole + w.slot, w.pmt, w.nt);
            // part lengths base, base + dk, base + 2 dk, ...; the last part also takes what the division leaves
            const int dk = p.k_stagger;
            const int base_len = (p.num_kb - dk * (ks * (ks - 1) / 2)) / ks;
            w.kb0 = w.part * base_len + dk * (w.part * (w.part - 1) / 2);
            w.kb1 = w.part + 1 == ks ? p.num_kb : w.kb0 + base_len + dk * w.part;
        }
        w.ncol0 = w.nt * BN;
        w.width = tile_n(w.nt);
        return w;
    };
    // Scheduler ring: the leader's producer lane takes list positions from the launch's counter and writes them
    // into the same slot of both CTAs; every reader acknowledges on the leader's "slot free" barrier.
    auto sched_ack = [&](int ss) { mbar_arrive_cluster(mapa_shared(sempty_bar(ss), 0)); };

    if (warp == 0) {
        // ---------------------------------------------------------------- scheduler (leader) + TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            long issued = 0;
            const uint64_t pol_a = make_policy(p.hint_a), pol_b = make_policy(p.hint_b);
            // Leader: take the next list position and publish it to both CTAs.  It runs one entry ahead of the
            // loads (the atomic's latency hides behind the copies of the current tile).
            bool exhausted = false;
            auto publish = [&]() -> int {
                if (exhausted) return -1;
                if (!mbar_wait_cluster(sempty_bar(ss), sphase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; return -1; }
                int t = atomicAdd(p.tile_counter, 1);
                if (t >= list_len) { t = -1; exhausted = true; }
                sched_slot[ss] = t;
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(sched_slot_addr + 4u * ss, 1)), "r"(t) : "memory");
                mbar_arrive(sfull_bar(ss));
                mbar_arrive_cluster(mapa_shared(sfull_bar(ss), 1));          // release.cluster: the peer sees its slot
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                return t;
            };
            int ahead = leader ? publish() : 0;
            while (ok) {
                int tile;
                if (leader) {
                    tile = ahead;
                    if (tile >= 0) ahead = publish();
                    if (!ok) break;
                } else {
                    if (!mbar_wait_cluster(sfull_bar(ss), sphase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    tile = sched_slot[ss];
                    sched_ack(ss);
                    if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                }
                if (tile < 0) break;
                const Work w = get_tile(tile);
                const int mt = 2 * w.pmt + static_cast<int>(rank);           // this CTA's 128-row tile
                const int bn0 = w.ncol0 + static_cast<int>(rank) * (w.width / 2);   // this CTA's half of the B tile
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    if (leader) mbar_arrive_expect_tx(full_bar(stage), 2 * Cfg::STAGE_BYTES);
                    const uint32_t bar = mapa_shared(full_bar(stage), 0);    // the leader's barrier
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    const bool drop = tile == 0 && kb - w.kb0 == p.drop_kb && ((p.drop_ranks >> rank) & 1);   // test hook
                    if (!drop) {
                        if (A_MN) tma2_load_3d(sa, &tmA, bar, 0, p.a_k0 + kb * BKE, (p.a_mn0 + mt * BM) >> CSH, pol_a);
                        else tma2_load_2d(sa, &tmA, bar, p.a_k0 + kb * BKE, p.a_mn0 + mt * BM, pol_a);
                        if (B_MN) tma2_load_3d(sb, &tmB, bar, 0, p.b_k0 + kb * BKE, (p.b_mn0 + bn0) >> CSH, pol_b);
                        else tma2_load_2d(sb, &tmB, bar, p.b_k0 + kb * BKE, p.b_mn0 + bn0, pol_b);
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if ((!ok || *abort_flag) && leader) {
                // Give-up path (the leader's barriers count both CTAs' bytes): let copies in flight land.
                const long back = issued < STAGES ? issued : STAGES;
                int s = stage; uint32_t ph = phase;
                for (long i = 0; i < back; ++i) {
                    if (--s < 0) { s = STAGES - 1; ph ^= 1u; }
                    unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(s), ph) && globaltimer_ns() - t0 < p.wait_limit_ns) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            for (int it = 0; ok;) {
                if (!mbar_wait(sfull_bar(ss), sphase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                const int tile = sched_slot[ss];
                sched_ack(ss);
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                const Work w = get_tile(tile);
                const uint32_t idesc = make_idesc(w.width, A_MN, B_MN, 2 * BM, TF32 ? 2u : 1u);
                const int ab = it & 1;
                const uint32_t aphase = (it >> 1) & 1u;
                if (!mbar_wait_cluster(tempty_bar(ab), aphase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + ab * ACC_STRIDE;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    // MN-major 32-bit operands: 32-byte swizzle units, whose pattern repeats every 4 k-rows (512 B)
                    constexpr uint64_t MN_LAYOUT = TF32 ? 1 : 2;
                    constexpr uint32_t MN_SBO = TF32 ? 512 : 1024;
                    const uint64_t adesc = A_MN ? make_smem_desc(sa, BKE * 128, MN_SBO, MN_LAYOUT) : make_smem_desc(sa, 16, 1024);
                    const uint64_t bdesc = B_MN ? make_smem_desc(sb, BKE * 128, MN_SBO, MN_LAYOUT) : make_smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int k = 0; k < BKE / UK; ++k) {
                        // K-major: UK elements = 32 B along the swizzled row; MN-major: UK k-rows of 128 B
                        const uint64_t aoff = static_cast<uint64_t>((A_MN ? k * UK * 128 : k * 32) >> 4);
                        const uint64_t boff = static_cast<uint64_t>((B_MN ? k * UK * 128 : k * 32) >> 4);
                        if (TF32) umma2_tf32(tmem_d, adesc + aoff, bdesc + boff, idesc, (kb > w.kb0 || k != 0) ? 1u : 0u);
                        else umma2_f16(tmem_d, adesc + aoff, bdesc + boff, idesc, (kb > w.kb0 || k != 0) ? 1u : 0u);
                    }
                    umma2_commit_both(empty_bar(stage));                     // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma2_commit_both(tfull_bar(ab));                    // accumulator ready in both CTAs
                ++it;
            }
            if (!ok || *abort_flag) {
                umma2_commit_local(drain_bar);
                unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(drain_bar, 0) && globaltimer_ns() - t0 < p.wait_limit_ns) {}
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps (both CTAs)
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        int ss = 0; uint32_t sphase = 0;
        bool ok = true;
        for (int it = 0; ok;) {
            int tile = -2;
            if (lane == 0) {
                if (mbar_wait_cluster(sfull_bar(ss), sphase, abort_flag, p.wait_limit_ns)) {
                    tile = sched_slot[ss];
                    sched_ack(ss);
                }
            }
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
            if (tile < 0) break;                                             // -1: list exhausted, -2: gave up
            const Work w = get_tile(tile);
            const int mt = 2 * w.pmt + static_cast<int>(rank);
            const int nt = w.nt;
            const int ab = it & 1;
            const uint32_t aphase = (it >> 1) & 1u;
            if (!mbar_wait(tfull_bar(ab), aphase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tmem_row = tmem_base + ab * ACC_STRIDE + (static_cast<uint32_t>(quad * 32) << 16);
            if (EPI == EPI_FOLD) epilogue_fold(p, mt, nt, row, tmem_row);
            else if (EPI == EPI_RESID && TF32) epilogue_resid_f32(p, &tmC, g_staging + (warp - 2) * 8192, mt, nt, row, lane, tmem_row);
            else if (EPI == EPI_RESID) epilogue_resid(p, &tmC, g_staging + (warp - 2) * 8192, mt, nt, row, lane, tmem_row);
            else {
                // parts of a split tile add in the order of their index: wait for this warp's rows of the part before
                int* flag = w.slot >= 0 ? p.split_flags + w.slot * 8 + static_cast<int>(rank) * 4 + quad : nullptr;
                if (w.part > 0) {
                    if (lane == 0 && !flag_wait_ge(flag, w.part, abort_flag, p.wait_limit_ns)) ok = false;
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                }
                epilogue_f32_tile(&tmC, g_staging + (warp - 2) * 8192, w.ncol0, p.c_row0 + mt * BM + quad * 32, lane, tmem_row,
                                  w.width, p.accumulate != 0 || w.part > 0);
                if (flag != nullptr && w.part + 1 < ks && lane == 0) {
                    bulk_wait_all();                                         // this warp's stores / additions are complete
                    flag_release(flag, w.part + 1);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(ab), 0));   // the leader owns this barrier
            ++it;
        }
        if (EPI != EPI_FOLD && lane == 0) bulk_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                          // no CTA leaves while its pair may still signal it or read its memory
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, VPCE_DEV_WAIT_EXPIRED);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem2_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------ small kernels
// Folds the per-tile partial states of one strip into the running per-token state (Eq. 2
// applied to two states: m = max(m1, m2), z = z1 e^{m1-m} + z2 e^{m2-m}), in tile order so the
// result does not depend on which CTA produced which tile.  On the last step it also emits
// lse = m + log z and loss = lse - y_t (Algorithm 3, output line).
__global__ void vpce_merge_kernel(const float* __restrict__ pm, const float* __restrict__ pz, int part_ld, int n_tiles,
                                  float* __restrict__ sm, float* __restrict__ sz, const float* __restrict__ ylab,
                                  int rows, int first, int last, const int32_t* __restrict__ labels, int ignore_index,
                                  int V, float* __restrict__ lse, float* __restrict__ loss, int* status) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= rows) return;
    float m = first ? NEG_INF : sm[n];
    float z = first ? 0.f : sz[n];
    for (int t = 0; t < n_tiles; ++t) {
        const float m2 = pm[static_cast<size_t>(t) * part_ld + n];
        const float z2 = pz[static_cast<size_t>(t) * part_ld + n];
        const float mn = fmaxf(m, m2);
        z = z * ex2f((m - mn) * LOG2E) + z2 * ex2f((m2 - mn) * LOG2E);   // m = -inf contributes 0
        m = mn;
    }
    if (!last) { sm[n] = m; sz[n] = z; return; }
    const float l = m + logf(z);
    lse[n] = l;
    const int t = labels[n];
    float out = 0.f;
    if (t != ignore_index) {
        if (static_cast<unsigned>(t) < static_cast<unsigned>(V)) out = l - ylab[n];
        else atomicOr(status, VPCE_DEV_LABEL_OUT_OF_RANGE);
    }
    loss[n] = out;
}

// One block: counts valid labels (fixed order) and stores 1 / n_valid (0 when there is none).
__global__ void vpce_count_valid_kernel(const int32_t* __restrict__ labels, long T, int V, int ignore_index,
                                        float* inv_n_valid, int* n_valid_out, int* status) {
    __shared__ int part[1024];
    int c = 0, bad = 0;
    for (long i = threadIdx.x; i < T; i += blockDim.x) {
        const int t = labels[i];
        if (t != ignore_index) {
            if (static_cast<unsigned>(t) < static_cast<unsigned>(V)) ++c; else bad = 1;
        }
    }
    if (bad && status) atomicOr(status, VPCE_DEV_LABEL_OUT_OF_RANGE);
    part[threadIdx.x] = c;
    __syncthreads();
    for (int s = blockDim.x / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (inv_n_valid) *inv_n_valid = part[0] > 0 ? 1.0f / static_cast<float>(part[0]) : 0.f;
        if (n_valid_out) *n_valid_out = part[0];
    }
}

// One block: masked mean of the per-token loss, double accumulation in a fixed order.
__global__ void vpce_mean_loss_kernel(const float* __restrict__ loss, const int32_t* __restrict__ labels, long T, int V,
                                      int ignore_index, float* mean_out, int* n_valid_out) {
    __shared__ double sums[1024];
    __shared__ int cnts[1024];
    double s = 0.0; int c = 0;
    for (long i = threadIdx.x; i < T; i += blockDim.x) {
        const int t = labels[i];
        if (t != ignore_index && static_cast<unsigned>(t) < static_cast<unsigned>(V)) { s += loss[i]; ++c; }
    }
    sums[threadIdx.x] = s; cnts[threadIdx.x] = c;
    __syncthreads();
    for (int k = blockDim.x / 2; k > 0; k >>= 1) {
        if (threadIdx.x < k) { sums[threadIdx.x] += sums[threadIdx.x + k]; cnts[threadIdx.x] += cnts[threadIdx.x + k]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        *mean_out = cnts[0] > 0 ? static_cast<float>(sums[0] / cnts[0]) : 0.f;
        *n_valid_out = cnts[0];
    }
}

// Gradient of the masked mean with respect to the per-token loss: upstream / n_valid on valid tokens, 0 elsewhere.
__global__ void vpce_mean_grad_kernel(const int32_t* __restrict__ labels, long T, int V, int ignore_index,
                                      const int* __restrict__ n_valid, const float* __restrict__ upstream,
                                      float* __restrict__ dloss) {
    const long i = static_cast<long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= T) return;
    const int nv = *n_valid;
    const float g = (upstream ? *upstream : 1.f) * (nv > 0 ? 1.0f / static_cast<float>(nv) : 0.f);
    const int t = labels[i];
    dloss[i] = (t != ignore_index && static_cast<unsigned>(t) < static_cast<unsigned>(V)) ? g : 0.f;
}

__global__ void vpce_clear_status_kernel(int* status) { if (threadIdx.x < 8) status[threadIdx.x] = 0; }

}  // namespace vpce
