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
#include "vp_ce_kernels.cuh"

namespace {

using namespace vpce;

// ------------------------------------------------------------------------------------ host side
std::atomic<long long> g_launches{0};

// Optional per-kernel timing: when enabled, every GEMM launch is bracketed by two events on the
// launching stream; vp_ce_profile_collect sums the elapsed times per kernel kind.
struct ProfEntry { int kind; cudaEvent_t a, b; };
std::mutex g_prof_mu;
bool g_prof_on = false;
std::vector<ProfEntry> g_prof;

// Limit of every wait inside the kernels (vp_ce_set_wait_limit_ns) and the one-shot test hook that makes the next
// launch of one kernel kind lose a copy (vp_ce_debug_drop_copy): kind in bits 0-7, k-block in bits 8-23, CTA ranks
// in bits 24-27; -1 = nothing armed.
std::atomic<unsigned long long> g_wait_limit_ns{kDefaultWaitLimitNs};
std::atomic<int> g_drop{-1};

// Fills the launch-time fields every GEMM launch shares.
GemmParams finish_params(const GemmParams& p, int epi) {
    GemmParams q = p;
    q.wait_limit_ns = g_wait_limit_ns.load(std::memory_order_relaxed);
    q.drop_kb = -1;
    q.drop_ranks = 0;
    int armed = g_drop.load(std::memory_order_relaxed);
    if (armed >= 0 && (armed & 0xff) == epi && g_drop.compare_exchange_strong(armed, -1)) {
        q.drop_kb = (armed >> 8) & 0xffff;
        q.drop_ranks = (armed >> 24) & 0xf;
    }
    return q;
}

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

bool ws_layout(int64_t T_chunk, int64_t d, int64_t block_v, WsLayout* L, int g_elem_bytes = 2) {
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
    L->G = off;       off = align_up(off + g_elem_bytes * static_cast<size_t>(T_chunk) * block_v, 1024);
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

// 2-D tensor map over a row-major [rows, cols] matrix of bf16 (elem_bytes 2) or fp32 (4): dim0 = cols
// (contiguous), 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld_elems, uint32_t box_cols,
              uint32_t box_rows, int elem_bytes = 2) {
    auto enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld_elems * elem_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUresult r = enc(map, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// MN-major operand of a row-major [k_rows, mn_cols] matrix (mn_cols % 64 == 0) as a 3-D tensor
// {64 contiguous elements, k_rows, mn_cols / 64}: one box {64, 64, chunks} per k-block lands in
// shared memory as `chunks` consecutive 64 x 128-byte blocks, the layout the MMA descriptor expects.
// (fp32: chunks of 32 elements and 32 k-rows per box.)
bool make_map_mn3d(CUtensorMap* map, const void* ptr, uint64_t k_rows, uint64_t mn_cols, uint64_t ld_elems, uint32_t chunks,
                   int elem_bytes = 2) {
    auto enc = get_encode();
    const uint64_t ce = 128 / elem_bytes;                 // elements per 128-byte chunk row = k-rows per stage
    if (!enc || mn_cols % ce) return false;
    cuuint64_t dims[3] = {ce, k_rows, mn_cols / ce};
    cuuint64_t strides[2] = {ld_elems * elem_bytes, 128};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(ce), static_cast<cuuint32_t>(ce), chunks};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType dt = elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    // MN-major 32-bit operands are swizzled in 32-byte units (what the tensor core expects for them)
    const CUtensorMapSwizzle sw = elem_bytes == 4 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
    CUresult r = enc(map, dt, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Per-device host-side caches are atomics: concurrent callers may both do the (idempotent) set-up, none reads
// a half-written value.
int num_sms() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cached[dev].load(std::memory_order_acquire);
    if (!n) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev].store(n, std::memory_order_release);
    }
    return n;
}

// Raises the dynamic shared-memory limit of `kern` once per device (the attribute is per device and function).
template <typename K>
cudaError_t ensure_smem_attr(K kern, int smem_bytes, std::atomic<bool>* done) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (!done[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        if (e != cudaSuccess) return e;
        done[dev].store(true, std::memory_order_release);
    }
    return cudaSuccess;
}

template <int BN, bool A_MN, bool B_MN, int EPI>
cudaError_t launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const GemmParams& p,
                        cudaStream_t st) {
    constexpr int SMEM = smem_total<BN, EPI>();
    auto kern = vpce_gemm_kernel<BN, A_MN, B_MN, EPI>;
    static std::atomic<bool> attr_set[64];
    if (cudaError_t e = ensure_smem_attr(kern, SMEM, attr_set); e != cudaSuccess) return e;
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
    kern<<<grid, NUM_THREADS, SMEM, st>>>(tmA, tmB, tmC, finish_params(p, EPI));
    if (prof) {
        cudaEventRecord(pe.b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.push_back(pe);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <int BN, bool A_MN, bool B_MN, int EPI, bool TF32 = false>
cudaError_t launch_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const GemmParams& p,
                        cudaStream_t st) {
    constexpr int SMEM = pair_smem_total<BN, EPI>();
    auto kern = vpce_gemm_pair_kernel<BN, A_MN, B_MN, EPI, TF32>;
    static std::atomic<bool> attr_set[64];
    if (cudaError_t e = ensure_smem_attr(kern, SMEM, attr_set); e != cudaSuccess) return e;
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
    kern<<<grid, NUM_THREADS, SMEM, st>>>(tmA, tmB, tmC, finish_params(p, EPI));
    if (prof) {
        cudaEventRecord(pe.b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.push_back(pe);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

// How many of the last tiles of a gradient GEMM to run as two 128-column halves: after the whole
// rounds R = tiles % pairs tiles are left; as halves they finish in about 0.56 tile times instead of
// one, provided the 2R halves fit into one round (a half costs a little more than half a tile: it
// re-loads A and uses only half of each B box).
int pick_n_cut(int pm_tiles, int n_tiles, int pairs) {
    const int R = pairs > 0 ? (pm_tiles * n_tiles) % pairs : 0;
    return (R > 0 && 2 * R <= pairs) ? R : 0;
}

// Which GEMMs run as CTA pairs (bit 0 strip kernels, bit 1 input-gradient, bit 2 weight-gradient).
// All of them by default; VPCE_PAIR in the environment overrides it for A/B measurements.
int pair_mask() {
    static const int mask = [] {
        const char* e = getenv("VPCE_PAIR");
        return e ? atoi(e) : 7;
    }();
    return mask;
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

// clear_status: whether the call starts by zeroing the device status word (the public entry points do; the
// backward half of vp_ce_fwd_bwd_host does not, so that what its forward half flagged is still there at the end).
static vpce_status forward_impl(const void* H, const void* W, const int32_t* labels, int64_t T, int64_t d, int64_t V,
                                int64_t block_v, int32_t ignore_index, float* loss, float* lse, int64_t T_chunk,
                                int64_t chunk_index_base, void* workspace, size_t workspace_bytes, void* stream,
                                bool clear_status) {
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

    if (clear_status) {
        vpce_clear_status_kernel<<<1, 32, 0, st>>>(status);
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
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

vpce_status vp_ce_forward(const void* H, const void* W, const int32_t* labels, int64_t T, int64_t d, int64_t V,
                          int64_t block_v, int32_t ignore_index, float* loss, float* lse, int64_t T_chunk,
                          int64_t chunk_index_base, void* workspace, size_t workspace_bytes, void* stream) {
    return forward_impl(H, W, labels, T, d, V, block_v, ignore_index, loss, lse, T_chunk, chunk_index_base, workspace,
                        workspace_bytes, stream, true);
}

static vpce_status backward_impl(const void* H, const void* W, const int32_t* labels, const float* lse,
                                 const float* dloss, void* dH, float* dW, int64_t T, int64_t d, int64_t V,
                                 int64_t block_v, int32_t ignore_index, int64_t T_chunk, int64_t chunk_index_base,
                                 int accumulate_dW, void* workspace, size_t workspace_bytes, void* stream,
                                 bool clear_status) {
    WsLayout L;
    if (T == 0) {                                                      // empty batch: dW gets no contribution
        if (!accumulate_dW && dW && V > 0 && d > 0 &&
            cudaMemsetAsync(dW, 0, static_cast<size_t>(V) * d * 4, static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return VPCE_CUDA_ERROR;
        return VPCE_OK;
    }
    if (!lse || (!dH && !dW)) return VPCE_INVALID_ARG;                 // either gradient may be left out, not both
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

    if (clear_status) {
        vpce_clear_status_kernel<<<1, 32, 0, st>>>(status);
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
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
            ph.dH = dH ? static_cast<__nv_bfloat16*>(dH) + tok0 * d : nullptr; ph.out_ld = static_cast<int>(d);
            ph.first = (i == 0); ph.last = (i == P - 1);
            ph.status = status;
            ph.b_3d = mn3d;
            ph.n_cut = pick_n_cut((ph.m_tiles + 1) / 2, ph.n_tiles, num_sms() / 2);
            apply_tuning(ph, EPI_DH);
            ph.tile_counter = counters.take();
            if (!dH) {
                // input gradient not wanted
            } else if ((pmask & 2) && pair_ok && ph.m_tiles >= 2) {
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
            if (!dW) continue;                                         // weight gradient not wanted
            pw.dW = dW + v_lo * d; pw.out_ld = static_cast<int>(d);
            pw.accumulate = (accumulate_dW != 0) || (c > 0);
            pw.status = status;
            pw.a_3d = mn3d; pw.b_3d = mn3d;
            pw.n_cut = pick_n_cut((pw.m_tiles + 1) / 2, pw.n_tiles, num_sms() / 2);
            apply_tuning(pw, EPI_DW);
            pw.tile_counter = counters.take();
            if ((pmask & 4) && pair_ok && pw.m_tiles >= 2) {
                if (launch_pair<256, true, true, EPI_DW>(tmG_mn, tmH_mn2, tmG_mn, pw, st) != cudaSuccess) return VPCE_CUDA_ERROR;
            } else if (launch_grad<true, true, EPI_DW>(bn, tmG_mn, tmH_mn, pw, st) != cudaSuccess) {
                return VPCE_CUDA_ERROR;
            }
        }
    }
    return counters.failed ? VPCE_CUDA_ERROR : VPCE_OK;
}

vpce_status vp_ce_backward(const void* H, const void* W, const int32_t* labels, const float* lse, const float* dloss,
                           void* dH, float* dW, int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                           int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW, void* workspace,
                           size_t workspace_bytes, void* stream) {
    return backward_impl(H, W, labels, lse, dloss, dH, dW, T, d, V, block_v, ignore_index, T_chunk, chunk_index_base,
                         accumulate_dW, workspace, workspace_bytes, stream, true);
}

vpce_status vp_ce_mean_loss(const float* loss, const int32_t* labels, int64_t T, int64_t V, int32_t ignore_index,
                            float* mean_out, int32_t* n_valid_out, void* stream) {
    if (!mean_out || !n_valid_out || T < 0 || V <= 0 || (T > 0 && (!loss || !labels))) return VPCE_INVALID_ARG;
    // T == 0 (an empty batch) gives mean 0 and n_valid 0, like the empty-batch rule of the other calls
    vpce_mean_loss_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(loss, labels, T, static_cast<int>(V),
                                                                           ignore_index, mean_out, n_valid_out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? VPCE_OK : VPCE_CUDA_ERROR;
}

vpce_status vp_ce_mean_loss_grad(const int32_t* labels, int64_t T, int64_t V, int32_t ignore_index,
                                 const int32_t* n_valid, const float* upstream, float* dloss_out, void* stream) {
    if (!n_valid || T < 0 || V <= 0 || (T > 0 && (!labels || !dloss_out))) return VPCE_INVALID_ARG;
    if (T == 0) return VPCE_OK;
    vpce_mean_grad_kernel<<<static_cast<unsigned>((T + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        labels, T, static_cast<int>(V), ignore_index, n_valid, upstream, dloss_out);
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

int64_t vp_ce_set_wait_limit_ns(int64_t ns) {
    const unsigned long long prev = g_wait_limit_ns.load(std::memory_order_relaxed);
    if (ns > 0) {
        unsigned long long v = static_cast<unsigned long long>(ns);
        if (v < 1000000ull) v = 1000000ull;                     // at least 1 ms: far longer than any copy is in flight
        if (v > 60000000000ull) v = 60000000000ull;
        g_wait_limit_ns.store(v, std::memory_order_relaxed);
    }
    return static_cast<int64_t>(prev);
}

vpce_status vp_ce_debug_drop_copy(int kernel_kind, int k_block, int cta_ranks) {
    if (kernel_kind < 0) { g_drop.store(-1, std::memory_order_relaxed); return VPCE_OK; }
    if (kernel_kind > 3 || k_block < 0 || k_block > 0xffff || cta_ranks <= 0 || cta_ranks > 3) return VPCE_INVALID_ARG;
    g_drop.store(kernel_kind | (k_block << 8) | (cta_ranks << 24), std::memory_order_relaxed);
    return VPCE_OK;
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
    // the status word keeps what the forward half flagged: it is cleared once, at the start of the whole pass
    s = backward_impl(H_dev, W, labels_dev, lse_dev, nullptr, dH_dev, dW, T, d, V, block_v, ignore_index, T_chunk,
                      chunk_index_base, accumulate_dW, workspace, workspace_bytes, stream, false);
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
    static std::atomic<bool> attr_set[64];
    if (ensure_smem_attr(kern, Cfg::SMEM_TOTAL, attr_set) != cudaSuccess) return VPCE_CUDA_ERROR;

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
            kern<<<grid, NUM_THREADS, Cfg::SMEM_TOTAL, st>>>(tmH, tmW, tmH, finish_params(p, EPI_FOLD));
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

#include "vp_ce_f32.inc"
