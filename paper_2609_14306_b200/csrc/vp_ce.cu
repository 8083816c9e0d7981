// Fused vocabulary projection + cross-entropy for sm_100a (B200).
//
// A warp-specialised, persistent tcgen05 GEMM kernel is instantiated with four epilogues:
//   FOLD   strip Y = H_c W_q^T  -> per-tile partial (max, sum-exp) + target logit   (Eq. 2)
//   RESID  the same strip       -> G = dloss (exp(Y - lse) - onehot) as bf16       (App. C)
//   DH     dH_c += G W_q        (contract over the shard's vocabulary)
//   DW     dW_q += G^T H_c      (contract over the chunk's tokens)
// Operands reach shared memory by TMA (128-byte swizzle), accumulators live in tensor
// memory (two buffers, so the epilogue of tile i overlaps the MMAs of tile i+1), and the
// logit strip never reaches global memory.
//
// Two variants of the kernel exist:
//   vpce_gemm_pair_kernel  two CTAs of a cluster share one 256 x 256 tile (tcgen05 cta_group::2);
//                          the default whenever a launch has at least two 128-row tiles;
//   vpce_gemm_kernel       one CTA per 128 x BN tile, tiles handed out by an atomic counter;
//                          used for narrow problems and by vp_ce_forward_static.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner,
// warps 2..5 = epilogue (one thread per accumulator row).
//
// Every wait on an mbarrier is bounded: when it runs out the CTA records
// VPCE_DEV_WAIT_EXPIRED in the workspace status word, all roles leave their loops, pending
// copies and MMAs are drained (bounded again), TMEM is freed and the kernel returns.

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <vector>

#include "vp_ce.h"

namespace {

constexpr int BM = 128;          // accumulator rows per tile (TMEM lanes)
constexpr int BK = 64;           // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int UMMA_K = 16;       // K per tcgen05.mma for 16-bit inputs
constexpr int BN_VOCAB = 256;    // vocabulary columns per strip tile
constexpr int NUM_THREADS = 192;
constexpr int SMEM_BUDGET = 200 * 1024;    // operand stages
constexpr int SMEM_EXTRA = 2048;           // barriers + alignment slack
constexpr int G_STAGING_BYTES = 4 * 2 * 4096;   // RESID: per epilogue warp two 32-row x 64-column bf16 boxes
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s per wait

enum Epilogue { EPI_FOLD = 0, EPI_RESID = 1, EPI_DH = 2, EPI_DW = 3 };

struct GemmParams {
    int m_tiles, n_tiles, num_kb;
    int a_3d, b_3d;                        // MN-major operand fetched as one 3-D box (64 x 64 x chunks) per k-block
    int hint_a, hint_b, hint_c;            // L2 eviction hints for A loads, B loads, C stores: 0 normal, 1 first, 2 last
    int n_cut;                             // pair kernel: full-width tiles run as two halves at the end of the list
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
    int g_ld;
    int g_rows;                            // rows of the G workspace (T_chunk)
    // DH
    float* acc;                            // [T_chunk][acc_ld] fp32 running dH of the chunk
    int acc_ld;
    __nv_bfloat16* dH;                     // chunk base, leading dimension out_ld
    int first, last;
    // DW
    float* dW;                             // shard base (row v_lo), leading dimension out_ld
    int accumulate;
    int out_ld;
    int* status;
    int* tile_counter;                     // zero before the launch; tiles are taken with atomicAdd
};

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// ---- cluster / CTA-pair (cta_group::2) primitives
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
// TMA loads of a CTA pair: data lands in the executing CTA, the byte count is credited to `bar`,
// which may live in the peer CTA (shared::cluster address).  No multicast.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                             uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void tmem2_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem2_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem2_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma2_commit_local(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Arrives (once the issuing thread's MMAs retire) on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}

__device__ __forceinline__ uint64_t make_policy(int kind) {
    uint64_t pol;
    if (kind == 1) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else if (kind == 2) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, uint32_t src, int c0, int c1, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor (sm_100 format), 128-byte swizzle.
//   K-major operand : rows of 64 bf16 (128 B); 8-row groups 1024 B apart (SBO); LBO unused.
//   MN-major operand: 64 K-rows of 64 MN elements (128 B) per box; boxes of successive
//                     64-element MN chunks LBO bytes apart; 8-K-row groups 1024 B apart (SBO).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;                      // descriptor version of sm_100
    d |= 2ull << 61;                      // SWIZZLE_128B
    return d;
}
// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128, N = bn.
__host__ __device__ constexpr uint32_t make_idesc(int bn, bool a_mn, bool b_mn, int m = BM) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn) << 15) |
           (static_cast<uint32_t>(b_mn) << 16) | (static_cast<uint32_t>(bn >> 3) << 17) |
           (static_cast<uint32_t>(m >> 4) << 24);
}

template <int BN> struct StageCfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (SMEM_BUDGET / STAGE_BYTES) > 8 ? 8 : (SMEM_BUDGET / STAGE_BYTES);
    static constexpr int SMEM_TOTAL = STAGES * STAGE_BYTES + SMEM_EXTRA;
    // the residual epilogue stages its bf16 tile in shared memory for TMA stores
    static constexpr int SMEM_TOTAL_STAGED = SMEM_TOTAL + G_STAGING_BYTES;
};
template <int BN, int EPI> constexpr int smem_total() {
    return EPI == 1 ? StageCfg<BN>::SMEM_TOTAL_STAGED : StageCfg<BN>::SMEM_TOTAL;
}

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
    const int lrel = label - (p.v_lo + nt * BN_VOCAB);          // target column relative to the tile
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

// ncol0: first output column of the tile; n_this: its width (columns beyond cols_valid are skipped).
__device__ __forceinline__ void epilogue_dh(const GemmParams& p, int mt, int ncol0, int row, uint32_t tmem_row, int n_this) {
    const int grow = mt * BM + row;
    const bool row_ok = grow < p.rows_valid;
#pragma unroll 1
    for (int c = 0; c < (n_this + 31) / 32; ++c) {
        float v[32];
        __syncwarp();
        tmem_ld32(tmem_row + c * 32, v);
        tmem_ld_wait();
        const int col0 = ncol0 + c * 32;
        if (row_ok) {
        float* arow = p.acc + static_cast<size_t>(grow) * p.acc_ld + col0;
        __nv_bfloat16* orow = p.dH + static_cast<size_t>(grow) * p.out_ld + col0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {                                  // 8 columns per step
            if (col0 + 8 * q >= p.cols_valid) break;                   // d is a multiple of 8
            float* x = v + 8 * q;
            if (!p.first) {
                const float4 a0 = *reinterpret_cast<const float4*>(arow + 8 * q);
                const float4 a1 = *reinterpret_cast<const float4*>(arow + 8 * q + 4);
                x[0] += a0.x; x[1] += a0.y; x[2] += a0.z; x[3] += a0.w;
                x[4] += a1.x; x[5] += a1.y; x[6] += a1.z; x[7] += a1.w;
            }
            if (p.last) {
                uint4 o;
                o.x = pack_bf16x2(x[0], x[1]); o.y = pack_bf16x2(x[2], x[3]);
                o.z = pack_bf16x2(x[4], x[5]); o.w = pack_bf16x2(x[6], x[7]);
                *reinterpret_cast<uint4*>(orow + 8 * q) = o;
            } else {
                *reinterpret_cast<float4*>(arow + 8 * q) = make_float4(x[0], x[1], x[2], x[3]);
                *reinterpret_cast<float4*>(arow + 8 * q + 4) = make_float4(x[4], x[5], x[6], x[7]);
            }
        }
        }
    }
}

__device__ __forceinline__ void epilogue_dw(const GemmParams& p, int mt, int ncol0, int row, uint32_t tmem_row, int n_this) {
    const int grow = mt * BM + row;                                    // vocabulary row within the shard
    const bool row_ok = grow < p.rows_valid;
#pragma unroll 1
    for (int c = 0; c < (n_this + 31) / 32; ++c) {
        float v[32];
        __syncwarp();
        tmem_ld32(tmem_row + c * 32, v);
        tmem_ld_wait();
        const int col0 = ncol0 + c * 32;
        if (row_ok) {
        float* orow = p.dW + static_cast<size_t>(grow) * p.out_ld + col0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {                                  // 4 columns per step
            if (col0 + 4 * q >= p.cols_valid) break;
            float4 x = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            if (p.accumulate) {
                const float4 a = *reinterpret_cast<const float4*>(orow + 4 * q);
                x.x += a.x; x.y += a.y; x.z += a.z; x.w += a.w;
            }
            *reinterpret_cast<float4*>(orow + 4 * q) = x;
        }
        }
    }
}

// ------------------------------------------------------------------------------------ the GEMM kernel
// Tiles are handed out dynamically: the producer lane takes the next tile index from a global
// counter (atomicAdd) and publishes it to the MMA lane and the epilogue warps through a small
// shared-memory ring guarded by mbarriers, so a CTA that finishes early simply takes more tiles.
// The last n-tile of a row may be narrower than BN (its MMA uses N = valid columns rounded up
// to 16), so an output width that is not a multiple of BN costs no padded tensor-core work.
constexpr int SCHED_DEPTH = 4;

template <int BN, bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
vpce_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
    using Cfg = StageCfg<BN>;
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
                if (!mbar_wait(sempty_bar(ss), sphase ^ 1u, abort_flag)) { ok = false; break; }
                int tile = atomicAdd(p.tile_counter, 1);
                if (tile >= total_tiles) tile = -1;
                sched_slot[ss] = tile;
                mbar_arrive(sfull_bar(ss));                              // release: the slot is visible to waiters
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int mt, nt;
                decode_tile(p, tile, mt, nt);
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(full_bar(stage), Cfg::STAGE_BYTES);
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    issue(mt, nt, kb, sa, sa + Cfg::A_BYTES, full_bar(stage));
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
                    while (!mbar_try_wait(full_bar(s), ph) && globaltimer_ns() - t0 < WAIT_LIMIT_NS) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            for (int it = 0; ok; ++it) {
                if (!mbar_wait(sfull_bar(ss), sphase, abort_flag)) { ok = false; break; }
                const int tile = sched_slot[ss];
                mbar_arrive(sempty_bar(ss));
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int mt, nt;
                decode_tile(p, tile, mt, nt);
                const uint32_t idesc = make_idesc(tile_n(nt), A_MN, B_MN);
                const int ab = it & 1;
                const uint32_t aphase = (it >> 1) & 1u;
                if (!mbar_wait(tempty_bar(ab), aphase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + ab * ACC_STRIDE;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
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
                while (!mbar_try_wait(drain_bar, 0) && globaltimer_ns() - t0 < WAIT_LIMIT_NS) {}
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
                if (mbar_wait(sfull_bar(ss), sphase, abort_flag)) {
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
            if (!mbar_wait(tfull_bar(ab), aphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tmem_row = tmem_base + ab * ACC_STRIDE + (static_cast<uint32_t>(quad * 32) << 16);
            if (EPI == EPI_FOLD) epilogue_fold(p, mt, nt, row, tmem_row);
            else if (EPI == EPI_RESID) epilogue_resid(p, &tmC, g_staging + (warp - 2) * 8192, mt, nt, row, lane, tmem_row);
            else if (EPI == EPI_DH) epilogue_dh(p, mt, nt * BN, row, tmem_row, tile_n(nt));
            else epilogue_dw(p, mt, nt * BN, row, tmem_row, tile_n(nt));
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(ab));
        }
        if (EPI == EPI_RESID && lane == 0) bulk_wait_all();             // staged stores have landed
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
// leader's "accumulator free" barrier.  Tiles are assigned round-robin to the pairs.
template <int BN> struct PairCfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = (BN / 2) * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (SMEM_BUDGET / STAGE_BYTES) > 8 ? 8 : (SMEM_BUDGET / STAGE_BYTES);
    static constexpr int SMEM_TOTAL = STAGES * STAGE_BYTES + SMEM_EXTRA;
};
template <int BN, int EPI> constexpr int pair_smem_total() {
    return PairCfg<BN>::SMEM_TOTAL + (EPI == 1 ? G_STAGING_BYTES : 0);
}

template <int BN, bool A_MN, bool B_MN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
vpce_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
    using Cfg = PairCfg<BN>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr uint32_t TMEM_COLS = 512u;
    constexpr uint32_t ACC_STRIDE = 256u;
    static_assert(BN == 256, "pair tiles are 256 x 256");

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
        constexpr int R = B_MN ? 128 : 32;
        return left >= BN ? BN : ((left + R - 1) / R * R);
    };
    // The work list, longest items first, handed out dynamically (greedy list scheduling):
    //   [0, n_whole)                  whole 256 x 256 tiles, n-fastest inside raster groups over the full-width n-tiles;
    //   [n_whole, n_whole + 2*n_cut)  the last n_cut full-width tiles as two 128-column halves each (gradient GEMMs
    //                                 only, and only when the host's estimate says the last round ends sooner that way);
    //   the rest                      the narrower last n-tile of every row, when the width is not a multiple of 256.
    constexpr bool kSplit = (EPI == EPI_DH || EPI == EPI_DW);
    const int n_wide = p.cols_valid / BN;                                    // full-width n-tiles per row
    const int n_wide_tiles = pm_tiles * n_wide;
    const int n_cut = kSplit ? min(p.n_cut, n_wide_tiles) : 0;              // chosen by the host (pick_n_cut)
    const int n_whole = n_wide_tiles - n_cut;
    const int n_tail = (p.n_tiles > n_wide) ? pm_tiles : 0;
    const int list_len = n_whole + 2 * n_cut + n_tail;
    auto decode_wide = [&](int tile, int& pmt, int& nt) {                    // raster order over the full-width n-tiles
        const int gn = min(p.group_n, max(n_wide, 1));
        const int per_group = gn * pm_tiles;
        const int g = tile / per_group;
        const int r = tile - g * per_group;
        const int n0 = g * gn;
        const int gw = min(gn, n_wide - n0);
        pmt = r / gw;
        nt = n0 + (r - pmt * gw);
    };
    auto get_tile = [&](int t, int& pmt, int& nt, int& ncol0, int& width) {
        if (t < n_whole) {
            decode_wide(t, pmt, nt);
            ncol0 = nt * BN; width = BN;
        } else if (t < n_whole + 2 * n_cut) {
            const int v = t - n_whole;
            decode_wide(n_whole + (v >> 1), pmt, nt);
            ncol0 = nt * BN + (v & 1) * (BN / 2); width = BN / 2;
        } else {
            pmt = t - (n_whole + 2 * n_cut);
            nt = n_wide;
            ncol0 = nt * BN; width = tile_n(nt);
        }
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
            while (ok) {
                int tile;
                if (leader) {
                    if (!mbar_wait_cluster(sempty_bar(ss), sphase ^ 1u, abort_flag)) { ok = false; break; }
                    tile = atomicAdd(p.tile_counter, 1);
                    if (tile >= list_len) tile = -1;
                    sched_slot[ss] = tile;
                    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(sched_slot_addr + 4u * ss, 1)), "r"(tile) : "memory");
                    mbar_arrive(sfull_bar(ss));
                    mbar_arrive_cluster(mapa_shared(sfull_bar(ss), 1));      // release.cluster: the peer sees its slot
                } else {
                    if (!mbar_wait_cluster(sfull_bar(ss), sphase, abort_flag)) { ok = false; break; }
                    tile = sched_slot[ss];
                    sched_ack(ss);
                }
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int pmt, nt, ncol0, width;
                get_tile(tile, pmt, nt, ncol0, width);
                const int mt = 2 * pmt + static_cast<int>(rank);             // this CTA's 128-row tile
                const int bn0 = ncol0 + static_cast<int>(rank) * (width / 2);   // this CTA's half of the B tile
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    if (leader) mbar_arrive_expect_tx(full_bar(stage), 2 * Cfg::STAGE_BYTES);
                    const uint32_t bar = mapa_shared(full_bar(stage), 0);    // the leader's barrier
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    if (A_MN) tma2_load_3d(sa, &tmA, bar, 0, p.a_k0 + kb * BK, (p.a_mn0 + mt * BM) >> 6, pol_a);
                    else tma2_load_2d(sa, &tmA, bar, p.a_k0 + kb * BK, p.a_mn0 + mt * BM, pol_a);
                    if (B_MN) tma2_load_3d(sb, &tmB, bar, 0, p.b_k0 + kb * BK, (p.b_mn0 + bn0) >> 6, pol_b);
                    else tma2_load_2d(sb, &tmB, bar, p.b_k0 + kb * BK, p.b_mn0 + bn0, pol_b);
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
                    while (!mbar_try_wait(full_bar(s), ph) && globaltimer_ns() - t0 < WAIT_LIMIT_NS) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int ss = 0; uint32_t sphase = 0;
            for (int it = 0; ok; ++it) {
                if (!mbar_wait(sfull_bar(ss), sphase, abort_flag)) { ok = false; break; }
                const int tile = sched_slot[ss];
                sched_ack(ss);
                if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
                if (tile < 0) break;
                int pmt, nt, ncol0, width;
                get_tile(tile, pmt, nt, ncol0, width);
                const uint32_t idesc = make_idesc(width, A_MN, B_MN, 2 * BM);
                const int ab = it & 1;
                const uint32_t aphase = (it >> 1) & 1u;
                if (!mbar_wait_cluster(tempty_bar(ab), aphase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + ab * ACC_STRIDE;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    const uint64_t adesc = A_MN ? make_smem_desc(sa, BK * 128, 1024) : make_smem_desc(sa, 16, 1024);
                    const uint64_t bdesc = B_MN ? make_smem_desc(sb, BK * 128, 1024) : make_smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t aoff = static_cast<uint64_t>((A_MN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        const uint64_t boff = static_cast<uint64_t>((B_MN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        umma2_f16(tmem_d, adesc + aoff, bdesc + boff, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma2_commit_both(empty_bar(stage));                     // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma2_commit_both(tfull_bar(ab));                    // accumulator ready in both CTAs
            }
            if (!ok || *abort_flag) {
                umma2_commit_local(drain_bar);
                unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(drain_bar, 0) && globaltimer_ns() - t0 < WAIT_LIMIT_NS) {}
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps (both CTAs)
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        int ss = 0; uint32_t sphase = 0;
        bool ok = true;
        for (int it = 0; ok; ++it) {
            int tile = -2;
            if (lane == 0) {
                if (mbar_wait_cluster(sfull_bar(ss), sphase, abort_flag)) {
                    tile = sched_slot[ss];
                    sched_ack(ss);
                }
            }
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (++ss == SCHED_DEPTH) { ss = 0; sphase ^= 1u; }
            if (tile < 0) break;                                             // -1: list exhausted, -2: gave up
            int pmt, nt, ncol0, width;
            get_tile(tile, pmt, nt, ncol0, width);
            const int mt = 2 * pmt + static_cast<int>(rank);
            const int ab = it & 1;
            const uint32_t aphase = (it >> 1) & 1u;
            if (!mbar_wait(tfull_bar(ab), aphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tmem_row = tmem_base + ab * ACC_STRIDE + (static_cast<uint32_t>(quad * 32) << 16);
            if (EPI == EPI_FOLD) epilogue_fold(p, mt, nt, row, tmem_row);
            else if (EPI == EPI_RESID) epilogue_resid(p, &tmC, g_staging + (warp - 2) * 8192, mt, nt, row, lane, tmem_row);
            else if (EPI == EPI_DH) epilogue_dh(p, mt, ncol0, row, tmem_row, width);
            else epilogue_dw(p, mt, ncol0, row, tmem_row, width);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(ab), 0));   // the leader owns this barrier
        }
        if (EPI == EPI_RESID && lane == 0) bulk_wait_all();
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

__global__ void vpce_clear_status_kernel(int* status) { if (threadIdx.x < 8) status[threadIdx.x] = 0; }

// ------------------------------------------------------------------------------------ host side
std::atomic<long long> g_launches{0};

// Optional per-kernel timing: when enabled, every GEMM launch is bracketed by two events on the
// launching stream; vp_ce_profile_collect sums the elapsed times per kernel kind.
struct ProfEntry { int kind; cudaEvent_t a, b; };
std::mutex g_prof_mu;
bool g_prof_on = false;
std::vector<ProfEntry> g_prof;

// Tile counters of the dynamic scheduler: one per launch, zeroed in bulk; a call that needs more
// launches than counters zeroes them again when it wraps (stream order makes that safe).
constexpr int NUM_TILE_COUNTERS = 1024;
struct CounterPool {
    int* base; int next; cudaStream_t st; bool failed;
    CounterPool(int* b, cudaStream_t s) : base(b), next(0), st(s), failed(false) {
        failed = cudaMemsetAsync(base, 0, 4 * NUM_TILE_COUNTERS, st) != cudaSuccess;
    }
    int* take() {
        if (next == NUM_TILE_COUNTERS) {
            failed = failed || cudaMemsetAsync(base, 0, 4 * NUM_TILE_COUNTERS, st) != cudaSuccess;
            next = 0;
        }
        return base + next++;
    }
};

struct WsLayout {
    size_t status, scalars, counters, sm, sz, ylab, pm, pz, G, acc, total;
};
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool ws_layout(int64_t T_chunk, int64_t d, int64_t block_v, WsLayout* L) {
    if (T_chunk <= 0 || d <= 0 || block_v <= 0) return false;
    if (T_chunk % BM || block_v % BN_VOCAB || d % 8) return false;
    if (T_chunk > (1 << 24) || block_v > (1 << 24) || d > (1 << 20)) return false;
    const size_t nt = static_cast<size_t>(block_v / BN_VOCAB);
    size_t off = 0;
    L->status = off;  off += 256;
    L->scalars = off; off += 256;
    L->counters = off; off += 4 * NUM_TILE_COUNTERS;
    L->sm = off;      off = align_up(off + 4 * T_chunk, 1024);
    L->sz = off;      off = align_up(off + 4 * T_chunk, 1024);
    L->ylab = off;    off = align_up(off + 4 * T_chunk, 1024);
    L->pm = off;      off = align_up(off + 4 * T_chunk * nt, 1024);
    L->pz = off;      off = align_up(off + 4 * T_chunk * nt, 1024);
    L->G = off;       off = align_up(off + 2 * static_cast<size_t>(T_chunk) * block_v, 1024);
    L->acc = off;     off = align_up(off + 4 * static_cast<size_t>(T_chunk) * d, 1024);
    L->total = off;
    return true;
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    });
    return fn;
}

// 2-D bf16 tensor map over a row-major [rows, cols] matrix: dim0 = cols (contiguous), 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld_elems, uint32_t box_cols,
              uint32_t box_rows) {
    auto enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld_elems * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// MN-major operand of a row-major [k_rows, mn_cols] matrix (mn_cols % 64 == 0) as a 3-D tensor
// {64 contiguous elements, k_rows, mn_cols / 64}: one box {64, 64, chunks} per k-block lands in
// shared memory as `chunks` consecutive 64 x 128-byte blocks, the layout the MMA descriptor expects.
bool make_map_mn3d(CUtensorMap* map, const void* ptr, uint64_t k_rows, uint64_t mn_cols, uint64_t ld_elems, uint32_t chunks) {
    auto enc = get_encode();
    if (!enc || mn_cols % 64) return false;
    cuuint64_t dims[3] = {64, k_rows, mn_cols / 64};
    cuuint64_t strides[2] = {ld_elems * 2, 128};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(BK), chunks};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int num_sms() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

template <int BN, bool A_MN, bool B_MN, int EPI>
cudaError_t launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const GemmParams& p,
                        cudaStream_t st) {
    constexpr int SMEM = smem_total<BN, EPI>();
    auto kern = vpce_gemm_kernel<BN, A_MN, B_MN, EPI>;
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int tiles = p.m_tiles * p.n_tiles;
    if (tiles <= 0 || p.num_kb <= 0) return cudaSuccess;
    const int grid = tiles < num_sms() ? tiles : num_sms();
    ProfEntry pe{EPI, nullptr, nullptr};
    bool prof = false;
    {
        std::lock_guard<std::mutex> lk(g_prof_mu);
        prof = g_prof_on;
    }
    if (prof && cudaEventCreate(&pe.a) == cudaSuccess && cudaEventCreate(&pe.b) == cudaSuccess) cudaEventRecord(pe.a, st);
    else prof = false;
    kern<<<grid, NUM_THREADS, SMEM, st>>>(tmA, tmB, tmC, p);
    if (prof) {
        cudaEventRecord(pe.b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.push_back(pe);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <int BN, bool A_MN, bool B_MN, int EPI>
cudaError_t launch_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const GemmParams& p,
                        cudaStream_t st) {
    constexpr int SMEM = pair_smem_total<BN, EPI>();
    auto kern = vpce_gemm_pair_kernel<BN, A_MN, B_MN, EPI>;
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int tiles = ((p.m_tiles + 1) / 2) * p.n_tiles;
    if (tiles <= 0 || p.num_kb <= 0) return cudaSuccess;
    const int max_pairs = num_sms() / 2;
    const int grid = 2 * (tiles < max_pairs ? tiles : max_pairs);
    ProfEntry pe{EPI, nullptr, nullptr};
    bool prof = false;
    {
        std::lock_guard<std::mutex> lk(g_prof_mu);
        prof = g_prof_on;
    }
    if (prof && cudaEventCreate(&pe.a) == cudaSuccess && cudaEventCreate(&pe.b) == cudaSuccess) cudaEventRecord(pe.a, st);
    else prof = false;
    kern<<<grid, NUM_THREADS, SMEM, st>>>(tmA, tmB, tmC, p);
    if (prof) {
        cudaEventRecord(pe.b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.push_back(pe);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

// How many of the full-width 256 x 256 tiles of a gradient GEMM to run as two 128-column halves.
// After the whole rounds, R = tiles % pairs full tiles and the narrow last-column tiles are left;
// greedy list scheduling of that remainder is simulated with and without cutting the R tiles
// (a half costs a little more than half a tile: it re-loads A and wastes half of each B box).
int pick_n_cut(int pm_tiles, int n_wide, int tail_width, int pairs) {
    const int wide = pm_tiles * n_wide;
    const int R = wide % pairs;
    if (R == 0 || pairs <= 0) return 0;
    const double half_cost = 0.56, tail_cost = tail_width > 0 ? 1.05 * tail_width / 256.0 : 0.0;
    const int n_tail = tail_width > 0 ? pm_tiles : 0;
    auto makespan = [&](int n_full, int n_half) {
        std::vector<double> load(pairs, 0.0);
        auto put = [&](double c) { *std::min_element(load.begin(), load.end()) += c; };
        for (int i = 0; i < n_full; ++i) put(1.0);
        for (int i = 0; i < n_half; ++i) put(half_cost);
        for (int i = 0; i < n_tail; ++i) put(tail_cost);
        return *std::max_element(load.begin(), load.end());
    };
    return makespan(0, 2 * R) + 0.02 < makespan(R, 0) ? R : 0;
}

// Which GEMMs run as CTA pairs (bit 0 strip kernels, bit 1 input-gradient, bit 2 weight-gradient).
// All of them by default; VPCE_PAIR in the environment overrides it for A/B measurements.
int pair_mask() {
    const char* e = getenv("VPCE_PAIR");
    return e ? atoi(e) : 7;
}

// Output-column tile for the two gradient GEMMs: 256 unless d is narrower; the last tile of a
// row runs with its own (narrower) MMA width, so d need not be a multiple of the tile.
int pick_bn(int64_t d) {
    if (d <= 64) return 64;
    if (d <= 128) return 128;
    if (d <= 192) return 192;
    return 256;
}

template <bool A_MN, bool B_MN, int EPI>
cudaError_t launch_grad(int bn, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p, cudaStream_t st) {
    switch (bn) {
        case 256: return launch_gemm<256, A_MN, B_MN, EPI>(tmA, tmB, tmA, p, st);
        case 192: return launch_gemm<192, A_MN, B_MN, EPI>(tmA, tmB, tmA, p, st);
        case 128: return launch_gemm<128, A_MN, B_MN, EPI>(tmA, tmB, tmA, p, st);
        default:  return launch_gemm<64, A_MN, B_MN, EPI>(tmA, tmB, tmA, p, st);
    }
}

// n-tiles per raster group: the B operand slice a group touches should stay L2-resident
// (<= ~48 MB), and groups are balanced.
int pick_group_n(int n_tiles, double b_total_bytes) {
    const double budget = 48.0 * 1024 * 1024;
    int groups = static_cast<int>((b_total_bytes + budget - 1) / budget);
    if (groups < 1) groups = 1;
    if (groups > n_tiles) groups = n_tiles;
    return (n_tiles + groups - 1) / groups;
}

// L2 eviction hints: the shard-side operand B is reused by every m-tile (keep it), the residual
// strip G is streamed out by RESID and streamed in by the two gradient GEMMs (let it go first).
void apply_tuning(GemmParams& p, int epi) {
    p.hint_a = 0;
    p.hint_b = 2;
    p.hint_c = (epi == EPI_RESID) ? 1 : 0;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

vpce_status check_common(const void* H, const void* W, const int32_t* labels, int64_t T, int64_t d, int64_t V,
                         int64_t block_v, int64_t T_chunk, int64_t chunk_index_base, const void* ws, size_t ws_bytes,
                         WsLayout* L) {
    if (!H || !W || !labels || !ws) return VPCE_INVALID_ARG;
    if (T <= 0 || d <= 0 || V <= 0 || block_v <= 0 || T_chunk <= 0 || chunk_index_base < 0) return VPCE_INVALID_ARG;
    if (!aligned16(H) || !aligned16(W) || !aligned16(ws)) return VPCE_UNSUPPORTED;
    if (T >= (1ll << 31) || V >= (1ll << 31)) return VPCE_UNSUPPORTED;
    if (!ws_layout(T_chunk, d, block_v, L)) return VPCE_UNSUPPORTED;
    if (ws_bytes < L->total) return VPCE_WORKSPACE_TOO_SMALL;
    return VPCE_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------ C ABI
extern "C" {

size_t vp_ce_workspace_bytes(int64_t T_chunk, int64_t d, int64_t block_v) {
    WsLayout L;
    return ws_layout(T_chunk, d, block_v, &L) ? L.total : 0;
}

const char* vp_ce_status_string(vpce_status s) {
    switch (s) {
        case VPCE_OK: return "ok";
        case VPCE_INVALID_ARG: return "invalid argument (null pointer or non-positive size)";
        case VPCE_UNSUPPORTED: return "unsupported (alignment, d % 8, block_v % 256 or T_chunk % 128)";
        case VPCE_WORKSPACE_TOO_SMALL: return "workspace too small";
        case VPCE_CUDA_ERROR: return "CUDA error";
        case VPCE_STATIC_SCRATCH_EXCEEDED:
            return "T_chunk * block_v too large for the built-in scratch of vp_ce_forward_static";
        default: return "unknown status";
    }
}

int64_t vp_ce_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

vpce_status vp_ce_forward(const void* H, const void* W, const int32_t* labels, int64_t T, int64_t d, int64_t V,
                          int64_t block_v, int32_t ignore_index, float* loss, float* lse, int64_t T_chunk,
                          int64_t chunk_index_base, void* workspace, size_t workspace_bytes, void* stream) {
    WsLayout L;
    if (T == 0) return VPCE_OK;                                        // empty batch: nothing to compute
    if (!loss || !lse) return VPCE_INVALID_ARG;
    vpce_status s = check_common(H, W, labels, T, d, V, block_v, T_chunk, chunk_index_base, workspace, workspace_bytes, &L);
    if (s != VPCE_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* sm = reinterpret_cast<float*>(ws + L.sm);
    float* sz = reinterpret_cast<float*>(ws + L.sz);
    float* ylab = reinterpret_cast<float*>(ws + L.ylab);
    float* pm = reinterpret_cast<float*>(ws + L.pm);
    float* pz = reinterpret_cast<float*>(ws + L.pz);

    CUtensorMap tmH, tmW, tmW_half;
    if (!make_map(&tmH, H, T, d, d, BK, BM) || !make_map(&tmW, W, V, d, d, BK, BN_VOCAB) ||
        !make_map(&tmW_half, W, V, d, d, BK, BN_VOCAB / 2))
        return VPCE_CUDA_ERROR;
    const bool pair_strip = (pair_mask() & 1) != 0;

    vpce_clear_status_kernel<<<1, 32, 0, st>>>(status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    CounterPool counters(reinterpret_cast<int*>(ws + L.counters), st);

    const int64_t P = (V + block_v - 1) / block_v;
    const int64_t n_chunks = (T + T_chunk - 1) / T_chunk;
    const int num_kb = static_cast<int>((d + BK - 1) / BK);
    for (int64_t c = 0; c < n_chunks; ++c) {
        const int64_t tok0 = c * T_chunk;
        const int rows = static_cast<int>((T - tok0) < T_chunk ? (T - tok0) : T_chunk);
        const int64_t cg = chunk_index_base + c;
        for (int64_t i = 0; i < P; ++i) {
            const int64_t q = ((cg - i) % P + P) % P;                  // Algorithm 3: q = (r - i) mod P
            const int64_t v_lo = q * block_v;
            const int cols = static_cast<int>((V - v_lo) < block_v ? (V - v_lo) : block_v);
            GemmParams p{};
            p.m_tiles = (rows + BM - 1) / BM;
            p.n_tiles = (cols + BN_VOCAB - 1) / BN_VOCAB;
            p.num_kb = num_kb;
            p.group_n = pick_group_n(p.n_tiles, 2.0 * cols * d);
            p.a_mn0 = static_cast<int>(tok0); p.a_k0 = 0;
            p.b_mn0 = static_cast<int>(v_lo); p.b_k0 = 0;
            p.rows_valid = rows; p.cols_valid = cols;
            p.v_lo = static_cast<int>(v_lo);
            p.labels = labels + tok0;
            p.ignore_index = ignore_index; p.V = static_cast<int>(V);
            p.pm = pm; p.pz = pz; p.ylab = ylab; p.part_ld = static_cast<int>(T_chunk);
            p.status = status;
            apply_tuning(p, EPI_FOLD);
            p.tile_counter = counters.take();
            if (pair_strip && p.m_tiles >= 2) {
                if (launch_pair<BN_VOCAB, false, false, EPI_FOLD>(tmH, tmW_half, tmH, p, st) != cudaSuccess) return VPCE_CUDA_ERROR;
            } else if (launch_gemm<BN_VOCAB, false, false, EPI_FOLD>(tmH, tmW, tmH, p, st) != cudaSuccess) {
                return VPCE_CUDA_ERROR;
            }
            vpce_merge_kernel<<<(rows + 255) / 256, 256, 0, st>>>(pm, pz, static_cast<int>(T_chunk), p.n_tiles, sm, sz, ylab,
                                                                  rows, i == 0, i == P - 1, labels + tok0, ignore_index,
                                                                  static_cast<int>(V), lse + tok0, loss + tok0, status);
            g_launches.fetch_add(1, std::memory_order_relaxed);
            if (cudaGetLastError() != cudaSuccess) return VPCE_CUDA_ERROR;
        }
    }
    return counters.failed ? VPCE_CUDA_ERROR : VPCE_OK;
}

vpce_status vp_ce_backward(const void* H, const void* W, const int32_t* labels, const float* lse, const float* dloss,
                           void* dH, float* dW, int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                           int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW, void* workspace,
                           size_t workspace_bytes, void* stream) {
    WsLayout L;
    if (T == 0) {                                                      // empty batch: dW gets no contribution
        if (!accumulate_dW && dW && V > 0 && d > 0 &&
            cudaMemsetAsync(dW, 0, static_cast<size_t>(V) * d * 4, static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return VPCE_CUDA_ERROR;
        return VPCE_OK;
    }
    if (!lse || !dH || !dW) return VPCE_INVALID_ARG;
    vpce_status s = check_common(H, W, labels, T, d, V, block_v, T_chunk, chunk_index_base, workspace, workspace_bytes, &L);
    if (s != VPCE_OK) return s;
    if (!aligned16(dH) || !aligned16(dW)) return VPCE_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* inv_n = reinterpret_cast<float*>(ws + L.scalars);
    __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(ws + L.G);
    float* acc = reinterpret_cast<float*>(ws + L.acc);

    CUtensorMap tmH_k, tmW_k, tmG_k, tmW_mn, tmG_mn, tmH_mn, tmG_st;
    if (!make_map(&tmG_st, G, T_chunk, block_v, block_v, 64, 32) ||
        !make_map(&tmH_k, H, T, d, d, BK, BM) || !make_map(&tmW_k, W, V, d, d, BK, BN_VOCAB) ||
        !make_map(&tmG_k, G, T_chunk, block_v, block_v, BK, BM) || !make_map(&tmW_mn, W, V, d, d, 64, BK) ||
        !make_map(&tmG_mn, G, T_chunk, block_v, block_v, 64, BK) || !make_map(&tmH_mn, H, T, d, d, 64, BK))
        return VPCE_CUDA_ERROR;

    vpce_clear_status_kernel<<<1, 32, 0, st>>>(status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    CounterPool counters(reinterpret_cast<int*>(ws + L.counters), st);
    if (!dloss) {
        vpce_count_valid_kernel<<<1, 1024, 0, st>>>(labels, T, static_cast<int>(V), ignore_index, inv_n, nullptr, status);
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }

    const int bn = pick_bn(d);
    // CTA-pair variants: half-width B boxes
    const int pmask = pair_mask();
    CUtensorMap tmW_khalf, tmW_mn2, tmH_mn2;
    const bool pair_ok = (bn == 256) && (d % 64 == 0);
    if (!make_map(&tmW_khalf, W, V, d, d, BK, BN_VOCAB / 2)) return VPCE_CUDA_ERROR;
    if (pair_ok && (!make_map_mn3d(&tmW_mn2, W, V, d, d, 2) || !make_map_mn3d(&tmH_mn2, H, T, d, d, 2))) return VPCE_CUDA_ERROR;
    // one-instruction fetch of MN-major operands when the contiguous extent is a multiple of 64
    const bool mn3d = (d % 64 == 0);
    if (mn3d) {
        if (!make_map_mn3d(&tmW_mn, W, V, d, d, bn / 64) || !make_map_mn3d(&tmH_mn, H, T, d, d, bn / 64) ||
            !make_map_mn3d(&tmG_mn, G, T_chunk, block_v, block_v, BM / 64))
            return VPCE_CUDA_ERROR;
    }
    const int64_t P = (V + block_v - 1) / block_v;
    const int64_t n_chunks = (T + T_chunk - 1) / T_chunk;
    for (int64_t c = 0; c < n_chunks; ++c) {
        const int64_t tok0 = c * T_chunk;
        const int rows = static_cast<int>((T - tok0) < T_chunk ? (T - tok0) : T_chunk);
        const int64_t cg = chunk_index_base + c;
        for (int64_t i = 0; i < P; ++i) {
            const int64_t q = ((cg - i) % P + P) % P;
            const int64_t v_lo = q * block_v;
            const int cols = static_cast<int>((V - v_lo) < block_v ? (V - v_lo) : block_v);
            const int strip_tiles_n = (cols + BN_VOCAB - 1) / BN_VOCAB;
            // (1) recompute the strip and form the residual G (bf16) in the workspace
            GemmParams p{};
            p.m_tiles = (rows + BM - 1) / BM;
            p.n_tiles = strip_tiles_n;
            p.num_kb = static_cast<int>((d + BK - 1) / BK);
            p.group_n = pick_group_n(p.n_tiles, 2.0 * cols * d);
            p.a_mn0 = static_cast<int>(tok0); p.b_mn0 = static_cast<int>(v_lo);
            p.rows_valid = rows; p.cols_valid = cols;
            p.v_lo = static_cast<int>(v_lo);
            p.labels = labels + tok0; p.lse = lse + tok0; p.dloss = dloss ? dloss + tok0 : nullptr;
            p.inv_n_valid = inv_n; p.ignore_index = ignore_index; p.V = static_cast<int>(V);
            p.G = G; p.g_ld = static_cast<int>(block_v); p.g_rows = static_cast<int>(T_chunk);
            p.status = status;
            apply_tuning(p, EPI_RESID);
            p.tile_counter = counters.take();
            if ((pmask & 1) && p.m_tiles >= 2) {
                if (launch_pair<BN_VOCAB, false, false, EPI_RESID>(tmH_k, tmW_khalf, tmG_st, p, st) != cudaSuccess) return VPCE_CUDA_ERROR;
            } else if (launch_gemm<BN_VOCAB, false, false, EPI_RESID>(tmH_k, tmW_k, tmG_st, p, st) != cudaSuccess) {
                return VPCE_CUDA_ERROR;
            }
            const int k_cols = strip_tiles_n * BN_VOCAB;               // columns of G written by step (1)
            const int m_rows = p.m_tiles * BM;                         // rows of G written by step (1)
            // (2) dH_c += G W_q : M = tokens, N = d, K = shard vocabulary
            GemmParams ph{};
            ph.m_tiles = p.m_tiles;
            ph.n_tiles = static_cast<int>((d + bn - 1) / bn);
            ph.num_kb = k_cols / BK;
            ph.group_n = pick_group_n(ph.n_tiles, 2.0 * k_cols * d);
            ph.a_mn0 = 0; ph.a_k0 = 0;
            ph.b_mn0 = 0; ph.b_k0 = static_cast<int>(v_lo);
            ph.rows_valid = rows; ph.cols_valid = static_cast<int>(d);
            ph.acc = acc; ph.acc_ld = static_cast<int>(d);
            ph.dH = static_cast<__nv_bfloat16*>(dH) + tok0 * d; ph.out_ld = static_cast<int>(d);
            ph.first = (i == 0); ph.last = (i == P - 1);
            ph.status = status;
            ph.b_3d = mn3d;
            ph.n_cut = pick_n_cut((ph.m_tiles + 1) / 2, static_cast<int>(d / 256), static_cast<int>(d % 256 ? ((d % 256 + 127) / 128 * 128) : 0), num_sms() / 2);
            apply_tuning(ph, EPI_DH);
            ph.tile_counter = counters.take();
            if ((pmask & 2) && pair_ok && ph.m_tiles >= 2) {
                if (launch_pair<256, false, true, EPI_DH>(tmG_k, tmW_mn2, tmG_k, ph, st) != cudaSuccess) return VPCE_CUDA_ERROR;
            } else if (launch_grad<false, true, EPI_DH>(bn, tmG_k, tmW_mn, ph, st) != cudaSuccess) {
                return VPCE_CUDA_ERROR;
            }
            // (3) dW_q += G^T H_c : M = shard vocabulary, N = d, K = chunk tokens
            GemmParams pw{};
            pw.m_tiles = (cols + BM - 1) / BM;
            pw.n_tiles = ph.n_tiles;
            pw.num_kb = m_rows / BK;
            pw.group_n = pick_group_n(pw.n_tiles, 2.0 * m_rows * d);
            pw.a_mn0 = 0; pw.a_k0 = 0;
            pw.b_mn0 = 0; pw.b_k0 = static_cast<int>(tok0);
            pw.rows_valid = cols; pw.cols_valid = static_cast<int>(d);
            pw.dW = dW + v_lo * d; pw.out_ld = static_cast<int>(d);
            pw.accumulate = (accumulate_dW != 0) || (c > 0);
            pw.status = status;
            pw.a_3d = mn3d; pw.b_3d = mn3d;
            pw.n_cut = pick_n_cut((pw.m_tiles + 1) / 2, static_cast<int>(d / 256), static_cast<int>(d % 256 ? ((d % 256 + 127) / 128 * 128) : 0), num_sms() / 2);
            apply_tuning(pw, EPI_DW);
            pw.tile_counter = counters.take();
            if ((pmask & 4) && pair_ok && pw.m_tiles >= 2) {
                if (launch_pair<256, true, true, EPI_DW>(tmG_mn, tmH_mn2, tmG_mn, pw, st) != cudaSuccess) return VPCE_CUDA_ERROR;
            } else if (launch_grad<true, true, EPI_DW>(bn, tmG_mn, tmH_mn, pw, st) != cudaSuccess) {
                return VPCE_CUDA_ERROR;
            }
        }
    }
    return VPCE_OK;
}

vpce_status vp_ce_mean_loss(const float* loss, const int32_t* labels, int64_t T, int64_t V, int32_t ignore_index,
                            float* mean_out, int32_t* n_valid_out, void* stream) {
    if (!loss || !labels || !mean_out || !n_valid_out || T <= 0 || V <= 0) return VPCE_INVALID_ARG;
    vpce_mean_loss_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(loss, labels, T, static_cast<int>(V),
                                                                           ignore_index, mean_out, n_valid_out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? VPCE_OK : VPCE_CUDA_ERROR;
}

vpce_status vp_ce_device_status(const void* workspace, int32_t* host_out, void* stream) {
    if (!workspace || !host_out) return VPCE_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host_out, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    return cudaStreamSynchronize(st) == cudaSuccess ? VPCE_OK : VPCE_CUDA_ERROR;
}

void vp_ce_profile_enable(int on) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = on != 0;
}

vpce_status vp_ce_profile_collect(double* ms_out, int64_t* launches_out) {
    if (!ms_out || !launches_out) return VPCE_INVALID_ARG;
    std::vector<ProfEntry> entries;
    {
        std::lock_guard<std::mutex> lk(g_prof_mu);
        entries.swap(g_prof);
    }
    for (int k = 0; k < 4; ++k) { ms_out[k] = 0.0; launches_out[k] = 0; }
    vpce_status rc = VPCE_OK;
    for (auto& e : entries) {
        float ms = 0.f;
        if (cudaEventSynchronize(e.b) == cudaSuccess && cudaEventElapsedTime(&ms, e.a, e.b) == cudaSuccess) {
            ms_out[e.kind] += ms;
            launches_out[e.kind] += 1;
        } else {
            rc = VPCE_CUDA_ERROR;
        }
        cudaEventDestroy(e.a);
        cudaEventDestroy(e.b);
    }
    return rc;
}

vpce_status vp_ce_fwd_bwd_host(const void* H_host, const int32_t* labels_host, const void* W, float* loss_host,
                               void* dH_host, float* dW, int64_t T, int64_t d, int64_t V, int64_t block_v,
                               int32_t ignore_index, int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW,
                               void* H_dev, int32_t* labels_dev, float* loss_dev, float* lse_dev, void* dH_dev,
                               void* workspace, size_t workspace_bytes, void* stream) {
    if (!H_host || !labels_host || !loss_host || !dH_host || !H_dev || !labels_dev || !loss_dev || !lse_dev || !dH_dev)
        return VPCE_INVALID_ARG;
    if (T <= 0 || d <= 0) return VPCE_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t hbytes = static_cast<size_t>(T) * d * 2;
    if (cudaMemcpyAsync(H_dev, H_host, hbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return VPCE_CUDA_ERROR;
    if (cudaMemcpyAsync(labels_dev, labels_host, static_cast<size_t>(T) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    vpce_status s = vp_ce_forward(H_dev, W, labels_dev, T, d, V, block_v, ignore_index, loss_dev, lse_dev, T_chunk,
                                  chunk_index_base, workspace, workspace_bytes, stream);
    if (s != VPCE_OK) return s;
    s = vp_ce_backward(H_dev, W, labels_dev, lse_dev, nullptr, dH_dev, dW, T, d, V, block_v, ignore_index, T_chunk,
                       chunk_index_base, accumulate_dW, workspace, workspace_bytes, stream);
    if (s != VPCE_OK) return s;
    if (cudaMemcpyAsync(loss_host, loss_dev, static_cast<size_t>(T) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    if (cudaMemcpyAsync(dH_host, dH_dev, hbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return VPCE_CUDA_ERROR;
    return cudaStreamSynchronize(st) == cudaSuccess ? VPCE_OK : VPCE_CUDA_ERROR;
}

// ------------------------------------------------------------------------------------ forward without a caller workspace
}  // extern "C"

namespace {

// Scratch of vp_ce_forward_static.  It is part of the loaded module: every GPU that loads this
// library holds these bytes until the process exits.  In host code the NAME of a __device__
// array is only a handle for the runtime, never an address a kernel may use; the device address
// is looked up once per device with cudaGetSymbolAddress and that pointer is what kernels get.
constexpr size_t STATIC_SCRATCH_BYTES = VPCE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

std::mutex g_static_mu;
unsigned char* g_static_ptr[64] = {nullptr};

// Device address of g_static_scratch on the current device (looked up on first use).
vpce_status static_scratch_address(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VPCE_CUDA_ERROR;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return VPCE_CUDA_ERROR;
        g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_ptr[dev];
    return VPCE_OK;
}

__global__ void vpce_copy_status_kernel(const int* status, int* out) { if (threadIdx.x == 0) *out = *status; }

}  // namespace

extern "C" {

vpce_status vp_ce_forward_static(const void* H, const void* W, const int32_t* labels, int64_t T, int64_t d, int64_t V,
                                 int64_t block_v, int32_t ignore_index, float* loss, float* lse, int64_t T_chunk,
                                 int64_t chunk_index_base, int32_t* device_status_out, void* stream) {
    if (!H || !W || !labels || !loss || !lse) return VPCE_INVALID_ARG;
    if (T <= 0 || d <= 0 || V <= 0 || block_v <= 0 || T_chunk <= 0 || chunk_index_base < 0) return VPCE_INVALID_ARG;
    if (!aligned16(H) || !aligned16(W)) return VPCE_UNSUPPORTED;
    if (T >= (1ll << 31) || V >= (1ll << 31)) return VPCE_UNSUPPORTED;
    WsLayout L;
    if (!ws_layout(T_chunk, d, block_v, &L)) return VPCE_UNSUPPORTED;
    // The forward touches the layout up to (not including) the residual strip G.
    if (L.G > STATIC_SCRATCH_BYTES) return VPCE_STATIC_SCRATCH_EXCEEDED;
    unsigned char* ws = nullptr;
    vpce_status s = static_scratch_address(&ws);
    if (s != VPCE_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* sm = reinterpret_cast<float*>(ws + L.sm);
    float* sz = reinterpret_cast<float*>(ws + L.sz);
    float* ylab = reinterpret_cast<float*>(ws + L.ylab);
    float* pm = reinterpret_cast<float*>(ws + L.pm);
    float* pz = reinterpret_cast<float*>(ws + L.pz);

    CUtensorMap tmH, tmW;
    if (!make_map(&tmH, H, T, d, d, BK, BM) || !make_map(&tmW, W, V, d, d, BK, BN_VOCAB)) return VPCE_CUDA_ERROR;
    using Cfg = StageCfg<BN_VOCAB>;
    auto kern = vpce_gemm_kernel<BN_VOCAB, false, false, EPI_FOLD>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_TOTAL) != cudaSuccess)
        return VPCE_CUDA_ERROR;

    // The array keeps whatever the previous call left: the status word must start at zero; the
    // running state is initialised by the first merge of every chunk and the partial slots are
    // fully rewritten before they are read.
    vpce_clear_status_kernel<<<1, 32, 0, st>>>(status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    CounterPool counters(reinterpret_cast<int*>(ws + L.counters), st);   // a memset, not an allocation

    const int64_t P = (V + block_v - 1) / block_v;
    const int64_t n_chunks = (T + T_chunk - 1) / T_chunk;
    const int num_kb = static_cast<int>((d + BK - 1) / BK);
    for (int64_t c = 0; c < n_chunks; ++c) {
        const int64_t tok0 = c * T_chunk;
        const int rows = static_cast<int>((T - tok0) < T_chunk ? (T - tok0) : T_chunk);
        const int64_t cg = chunk_index_base + c;
        for (int64_t i = 0; i < P; ++i) {
            const int64_t q = ((cg - i) % P + P) % P;
            const int64_t v_lo = q * block_v;
            const int cols = static_cast<int>((V - v_lo) < block_v ? (V - v_lo) : block_v);
            GemmParams p{};
            p.m_tiles = (rows + BM - 1) / BM;
            p.n_tiles = (cols + BN_VOCAB - 1) / BN_VOCAB;
            p.num_kb = num_kb;
            p.group_n = pick_group_n(p.n_tiles, 2.0 * cols * d);
            p.a_mn0 = static_cast<int>(tok0); p.b_mn0 = static_cast<int>(v_lo);
            p.rows_valid = rows; p.cols_valid = cols;
            p.v_lo = static_cast<int>(v_lo);
            p.labels = labels + tok0;
            p.ignore_index = ignore_index; p.V = static_cast<int>(V);
            p.pm = pm; p.pz = pz; p.ylab = ylab; p.part_ld = static_cast<int>(T_chunk);
            p.status = status;
            apply_tuning(p, EPI_FOLD);
            p.tile_counter = counters.take();
            const int tiles = p.m_tiles * p.n_tiles;
            const int grid = tiles < num_sms() ? tiles : num_sms();
            kern<<<grid, NUM_THREADS, Cfg::SMEM_TOTAL, st>>>(tmH, tmW, tmH, p);
            vpce_merge_kernel<<<(rows + 255) / 256, 256, 0, st>>>(pm, pz, static_cast<int>(T_chunk), p.n_tiles, sm, sz, ylab,
                                                                  rows, i == 0, i == P - 1, labels + tok0, ignore_index,
                                                                  static_cast<int>(V), lse + tok0, loss + tok0, status);
            g_launches.fetch_add(2, std::memory_order_relaxed);
            if (cudaGetLastError() != cudaSuccess) return VPCE_CUDA_ERROR;
        }
    }
    if (device_status_out) {
        vpce_copy_status_kernel<<<1, 32, 0, st>>>(status, device_status_out);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return VPCE_CUDA_ERROR;
    }
    return VPCE_OK;
}

}  // extern "C"
