// Exact one-hot terms of the two gradients.
//
// The residual strip G = dloss (softmax - onehot) is staged as bf16.  For all entries but one per token that rounding
// is random and averages out in the contractions; the target entry dloss (p_t - 1) is ~-dloss for every token, so its
// rounding error (up to 2^-9 relative, about sqrt(V) / 512 of the whole softmax part) has the same sign whenever dloss
// is the same number.  The residual epilogue therefore records, per token, delta_n = exact - rounded of that one
// entry (fp32), and the two kernels here add what the GEMMs missed:
//     dX[n, :]   += delta_n W[t_n, :]          (row-wise, one CTA per token)
//     dW[t_n, :] += delta_n X[n, :]            (a scatter; made deterministic by sorting the tokens by target)
// Sums run in a fixed order (token index within a target), so results stay bitwise reproducible.
#pragma once

#include "vp_ce_kernels.cuh"

namespace vpce {

constexpr int SORT_MAX = 16384;     // tokens one CTA sorts in shared memory (128 KB of 64-bit keys)
constexpr int FIX_SEG = 64;         // sorted positions per CTA of the scatter kernel
constexpr unsigned long long KEY_INVALID = ~0ull;

// Sorts the tokens of each sub-chunk of SORT_MAX tokens by (target, token index): key = target << 32 | index within
// the chunk; ignored or out-of-range targets get KEY_INVALID | index and end up last.  Keys are unique, so the sorted
// position of a key is simply the number of smaller keys: every thread counts that for one token against all keys of
// its sub-chunk (streamed through shared memory) and stores its key there.  n^2 comparisons, but all of them
// independent: ~30 us for 16384 tokens spread over the whole GPU, where a one-CTA sorting network took 170 us.
constexpr int RANK_TOKENS = 128;    // tokens per CTA
constexpr int RANK_PARTS = 4;       // threads per token: each counts against a quarter of every tile
constexpr int RANK_TILE = 2048;
__device__ __forceinline__ unsigned long long target_key(const int32_t* labels, int i, int ignore_index, int V) {
    const int t = labels[i];
    const unsigned long long hi = (t != ignore_index && static_cast<unsigned>(t) < static_cast<unsigned>(V))
                                      ? static_cast<unsigned long long>(static_cast<unsigned>(t)) : 0xFFFFFFFFull;
    return (hi << 32) | static_cast<unsigned>(i);
}
__global__ void __launch_bounds__(RANK_TOKENS * RANK_PARTS)
vpce_sort_targets_kernel(const int32_t* __restrict__ labels, int rows, int ignore_index, int V,
                         unsigned long long* __restrict__ keys) {
    __shared__ unsigned long long tile[RANK_TILE];
    __shared__ int part_rank[RANK_PARTS][RANK_TOKENS];
    const int blocks_per_sub = SORT_MAX / RANK_TOKENS;
    const int sub = blockIdx.x / blocks_per_sub;
    const int r0 = sub * SORT_MAX;
    const int n = min(SORT_MAX, rows - r0);
    const int tok0 = (blockIdx.x - sub * blocks_per_sub) * RANK_TOKENS;
    if (tok0 >= n) return;                                              // whole block past the end of the sub-chunk
    const int lane_tok = threadIdx.x % RANK_TOKENS, part = threadIdx.x / RANK_TOKENS;
    const int i = tok0 + lane_tok;                                      // token within the sub-chunk
    const bool mine = i < n;
    const unsigned long long key = mine ? target_key(labels, r0 + i, ignore_index, V) : 0ull;
    int rank = 0;
    for (int t0 = 0; t0 < n; t0 += RANK_TILE) {
        const int tn = min(RANK_TILE, n - t0);
        __syncthreads();
        for (int j = threadIdx.x; j < tn; j += blockDim.x) tile[j] = target_key(labels, r0 + t0 + j, ignore_index, V);
        __syncthreads();
        const int j0 = part * (RANK_TILE / RANK_PARTS), j1 = min(tn, j0 + RANK_TILE / RANK_PARTS);
#pragma unroll 8
        for (int j = j0; j < j1; ++j) rank += tile[j] < key ? 1 : 0;
    }
    part_rank[part][lane_tok] = rank;
    __syncthreads();
    if (part == 0 && mine) {
#pragma unroll
        for (int q = 1; q < RANK_PARTS; ++q) rank += part_rank[q][lane_tok];
        keys[r0 + rank] = key;
    }
}

// One pass over the fp32 input-gradient accumulator of a batch, one CTA per token row (row pitch d, d % 8 == 0):
//   Wr  != null: acc[n, :] += delta[n] * Wr[t_n - v0, :] for every token whose (valid) target lies in [v0, v0 + nv)
//                (Wr points at row v0 of the weight);
//   out != null: the row (with that term) is rounded to bf16 and written to out[n, :], acc is left as it was;
//   out == null: the row is written back to acc.
__global__ void __launch_bounds__(128)
vpce_finish_dx_kernel(float* __restrict__ acc, __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ Wr,
                      const int32_t* __restrict__ labels, const float* __restrict__ delta, int d, int v0, int nv,
                      int ignore_index) {
    const int n = blockIdx.x;
    float dl = 0.f;
    const __nv_bfloat16* wrow = nullptr;
    if (Wr) {
        const int t = labels[n];
        if (t != ignore_index && static_cast<unsigned>(t - v0) < static_cast<unsigned>(nv)) {
            dl = delta[n];
            wrow = Wr + static_cast<size_t>(t - v0) * d;
        }
    }
    if (!out && dl == 0.f) return;                            // nothing to add and nothing to convert
    float* arow = acc + static_cast<size_t>(n) * d;
    for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
        float4 a0 = __ldcs(reinterpret_cast<const float4*>(arow + c));
        float4 a1 = __ldcs(reinterpret_cast<const float4*>(arow + c + 4));
        if (dl != 0.f) {
            const uint4 w = *reinterpret_cast<const uint4*>(wrow + c);
            const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&w);
            const float2 w0 = __bfloat1622float2(wp[0]), w1 = __bfloat1622float2(wp[1]);
            const float2 w2 = __bfloat1622float2(wp[2]), w3 = __bfloat1622float2(wp[3]);
            a0.x = fmaf(dl, w0.x, a0.x); a0.y = fmaf(dl, w0.y, a0.y); a0.z = fmaf(dl, w1.x, a0.z); a0.w = fmaf(dl, w1.y, a0.w);
            a1.x = fmaf(dl, w2.x, a1.x); a1.y = fmaf(dl, w2.y, a1.y); a1.z = fmaf(dl, w3.x, a1.z); a1.w = fmaf(dl, w3.y, a1.w);
        }
        if (out) {
            uint4 o;
            o.x = pack_bf16x2(a0.x, a0.y); o.y = pack_bf16x2(a0.z, a0.w);
            o.z = pack_bf16x2(a1.x, a1.y); o.w = pack_bf16x2(a1.z, a1.w);
            *reinterpret_cast<uint4*>(out + static_cast<size_t>(n) * d + c) = o;
        } else {
            *reinterpret_cast<float4*>(arow + c) = a0;
            *reinterpret_cast<float4*>(arow + c + 4) = a1;
        }
    }
}

// First position of the sorted keys[0, n) whose key is >= x, found by all 256 threads of the CTA together: two steps of
// parallel probes (every 64th key, then the 64 keys of the bracket) instead of a 14-step dependent chain.
__device__ __forceinline__ int block_lower_bound(const unsigned long long* keys, int n, unsigned long long x, int* s_tmp) {
    if (threadIdx.x == 0) *s_tmp = n;
    __syncthreads();
    // step 1: the first probe position p = 64 k (k = 0 .. 255, + tail) with keys[p] >= x
    for (int p = threadIdx.x * 64; p < n; p += 256 * 64)
        if (keys[p] >= x) atomicMin(s_tmp, p);
    __syncthreads();
    const int hi = *s_tmp;                                   // keys[hi] >= x (or hi == n); the answer lies in (hi - 64, hi]
    __syncthreads();
    const int lo = max(0, hi - 63);
    const int q = lo + static_cast<int>(threadIdx.x);
    if (threadIdx.x < 64 && q < hi && keys[q] >= x) atomicMin(s_tmp, q);
    __syncthreads();
    const int r = *s_tmp;
    __syncthreads();
    return r;
}

// dWr[t - v0, :] += sum over the tokens n of one sorted sub-chunk with target t in [v0, v0 + nv) of delta[n] X[n, :].
//   keys      the sub-chunk's sorted keys (n of them); the tokens of a target form one run of consecutive positions
//   X, delta  point at the CHUNK's first token (keys carry indices within the chunk); X has row pitch d
//   dWr       points at row v0 of the weight gradient (row pitch d)
// Two launches with the same grid (segments of FIX_SEG positions, column blocks of 256), one thread per column.
// Pass 1 walks a segment's positions in order: a run that lies inside the segment is added to dWr by that CTA (the
// only writer of that row and column); a run that continues into a neighbouring segment leaves its partial sum in
// `partials` ([segment][2][d]: slot 0 = the segment's first run, slot 1 = a later run).  Pass 2: the CTA of the
// segment in which such a run ENDS adds the run's partial sums up from its first segment on and adds the total to dWr.
// Hence every sum has a fixed order whatever the scheduling.
__global__ void __launch_bounds__(256)
vpce_onehot_dw_kernel(const unsigned long long* __restrict__ keys, int n, const __nv_bfloat16* __restrict__ X,
                      const float* __restrict__ delta, int d, int v0, int nv, float* __restrict__ dWr,
                      float* __restrict__ partials) {
    __shared__ int s_tmp;
    __shared__ unsigned long long s_keys[FIX_SEG + 2];
    const int lo_pos = block_lower_bound(keys, n, static_cast<unsigned long long>(static_cast<unsigned>(v0)) << 32, &s_tmp);
    const int hi_pos = block_lower_bound(keys, n, static_cast<unsigned long long>(static_cast<unsigned>(v0 + nv)) << 32, &s_tmp);
    const int seg = blockIdx.x;
    const int col = blockIdx.y * 256 + threadIdx.x;
    const bool active = col < d;
    const int p0 = lo_pos + seg * FIX_SEG;
    if (p0 >= hi_pos) return;
    const int p1 = min(hi_pos, p0 + FIX_SEG);
    // keys of positions p0-1 .. p1 (neighbours outside [lo_pos, hi_pos) count as "another target")
    for (int i = threadIdx.x; i < p1 - p0 + 2; i += blockDim.x) {
        const int p = p0 - 1 + i;
        s_keys[i] = (p >= lo_pos && p < hi_pos) ? keys[p] : KEY_INVALID;
    }
    __syncthreads();
    const int left_label = static_cast<int>(s_keys[0] >> 32);
    float sum = 0.f;
    int run_start = p0;
    float term[8];                                                              // delta * x of 8 positions at a time:
    for (int p = p0; p < p1; ++p) {                                             // the gathers overlap, the sum stays in order
        if (((p - p0) & 7) == 0) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                term[u] = 0.f;
                if (active && p + u < p1) {
                    const unsigned iu = static_cast<unsigned>(s_keys[p + u - p0 + 1]);
                    term[u] = delta[iu] * __bfloat162float(X[static_cast<size_t>(iu) * d + col]);
                }
            }
        }
        const int label = static_cast<int>(s_keys[p - p0 + 1] >> 32);
        float tv = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) if (((p - p0) & 7) == u) tv = term[u];
        sum += tv;
        const int next_label = static_cast<int>(s_keys[p - p0 + 2] >> 32);     // position p + 1 (or the right neighbour)
        if (p + 1 == p1 || next_label != label) {                               // the run ends here, or the segment does
            const bool cont_left = run_start == p0 && left_label == label;
            const bool cont_right = p + 1 == p1 && next_label == label;
            if (active) {
                // the only contribution to this element in this launch, so the result does not depend on timing; issued
                // as a reduction (no value comes back), which keeps the walk from waiting for memory at every run
                if (!cont_left && !cont_right) atomicAdd(dWr + static_cast<size_t>(label - v0) * d + col, sum);
                else partials[(static_cast<size_t>(seg) * 2 + (run_start == p0 ? 0 : 1)) * d + col] = sum;
            }
            sum = 0.f;
            run_start = p + 1;
        }
    }
}

__global__ void __launch_bounds__(256)
vpce_onehot_dw_combine_kernel(const unsigned long long* __restrict__ keys, int n, int d, int v0, int nv,
                              float* __restrict__ dWr, const float* __restrict__ partials) {
    __shared__ int s_tmp;
    const int lo_pos = block_lower_bound(keys, n, static_cast<unsigned long long>(static_cast<unsigned>(v0)) << 32, &s_tmp);
    const int hi_pos = block_lower_bound(keys, n, static_cast<unsigned long long>(static_cast<unsigned>(v0 + nv)) << 32, &s_tmp);
    const int seg = blockIdx.x;
    const int q0 = lo_pos + seg * FIX_SEG;
    if (q0 >= hi_pos || seg == 0) return;                    // a run can only END here if it came in from a segment before
    const int q1 = min(hi_pos, q0 + FIX_SEG);
    const int label = static_cast<int>(keys[q0] >> 32);      // target of this segment's first run
    if (static_cast<int>(keys[q0 - 1] >> 32) != label) return;                                  // did not come in from the left
    const bool single = static_cast<int>(keys[q1 - 1] >> 32) == label;
    if (single && q1 < hi_pos && static_cast<int>(keys[q1] >> 32) == label) return;             // goes on to the right
    // the run ends in this segment: where did it start?
    const int start = block_lower_bound(keys, n, static_cast<unsigned long long>(static_cast<unsigned>(label)) << 32, &s_tmp);
    const int head = (start - lo_pos) / FIX_SEG;
    const int col = blockIdx.y * 256 + threadIdx.x;
    if (col >= d) return;
    // partial sums of segments head .. seg, in that order: the head's lies in slot 1 unless the run opens its segment
    float sum = __ldcg(partials + (static_cast<size_t>(head) * 2 + (start == lo_pos + head * FIX_SEG ? 0 : 1)) * d + col);
    for (int t = head + 1; t <= seg; t += 8) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (t + u <= seg) ? __ldcg(partials + static_cast<size_t>(t + u) * 2 * d + col) : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) if (t + u <= seg) sum += v[u];
    }
    atomicAdd(dWr + static_cast<size_t>(label - v0) * d + col, sum);      // again the element's only contribution
}

}  // namespace vpce
