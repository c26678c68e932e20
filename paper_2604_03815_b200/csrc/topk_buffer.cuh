// Per-row running top-k state shared by the score kernels (Algorithm 1 line 3, RowwiseTopK).
//
// A candidate is one 64-bit key: the high word is the score mapped to an unsigned integer that
// orders like the float, the low word is (2^32-1 - key index).  Larger key == better candidate
// under the library's ordering (score descending, index ascending), and all keys are distinct,
// so "the k largest keys" is exactly the required selection including its tie-break.
//
// A row owns CAP = 32*E slots in shared memory: slots [0,k) hold the current best k, sorted
// descending (0 = empty), slots [k, CAP) are an append-only pending area.  A score is appended
// only if it beats the row's threshold tau (the k-th best at the last compaction, -inf before k
// candidates exist).  Because keys are visited in increasing index order, a score equal to tau
// can never displace a kept key, so the strict comparison loses nothing.  When the pending area
// is nearly full a warp sorts the row's CAP slots cooperatively and keeps the first k.
#pragma once

#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace kmip {

typedef unsigned long long cand_t;

__device__ __forceinline__ uint32_t order_bits(float s) {
    const uint32_t u = __float_as_uint(s);
    return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);  // negative: flip all bits; else set the sign bit
}
__device__ __forceinline__ float unorder_bits(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}
__device__ __forceinline__ cand_t make_cand(float s, int idx) {
    s += 0.0f;  // -0.0 -> +0.0 so that equal scores have equal high words
    return ((cand_t)order_bits(s) << 32) | (cand_t)(0xFFFFFFFFu - (uint32_t)idx);
}
__device__ __forceinline__ int cand_index(cand_t c) { return (int)(0xFFFFFFFFu - (uint32_t)c); }
__device__ __forceinline__ float cand_score(cand_t c) { return unorder_bits((uint32_t)(c >> 32)); }

__device__ __forceinline__ cand_t cmax(cand_t a, cand_t b) { return a > b ? a : b; }
__device__ __forceinline__ cand_t cmin(cand_t a, cand_t b) { return a > b ? b : a; }

// Bitonic sort, descending, of 32*E keys held E per lane; element g = e*32 + lane.
template <int E>
__device__ __forceinline__ void warp_sort_desc(cand_t (&v)[E], int lane) {
    constexpr int CAP = 32 * E;
#pragma unroll
    for (int kk = 2; kk <= CAP; kk <<= 1) {
#pragma unroll
        for (int j = kk >> 1; j > 0; j >>= 1) {
            if (j >= 32) {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const int pe = e ^ (j >> 5);
                    if (pe > e) {
                        const bool desc = ((e * 32) & kk) == 0;
                        const cand_t a = v[e], b = v[pe];
                        const cand_t mx = cmax(a, b), mn = cmin(a, b);
                        v[e] = desc ? mx : mn;
                        v[pe] = desc ? mn : mx;
                    }
                }
            } else {
                const bool lower = (lane & j) == 0;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const bool desc = (((e * 32) | lane) & kk) == 0;
                    const cand_t o = __shfl_xor_sync(0xFFFFFFFFu, v[e], j);
                    v[e] = (lower == desc) ? cmax(v[e], o) : cmin(v[e], o);
                }
            }
        }
    }
}

// Warp-cooperative compaction of one row: sort slots [0, k+cnt), keep the best k in [0,k),
// return the new threshold (score of the k-th best, -inf while fewer than k candidates exist).
// All 32 lanes call it with the same arguments; the caller's earlier writes to `row` must be
// visible (a __syncwarp() precedes the reads here).
template <int E>
__device__ __forceinline__ float warp_compact_row(cand_t* row, int k, int cnt, int lane) {
    __syncwarp();
    cand_t v[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int g = e * 32 + lane;
        v[e] = (g < k + cnt) ? row[g] : 0ull;
    }
    warp_sort_desc<E>(v, lane);
    __syncwarp();
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int g = e * 32 + lane;
        if (g < k) row[g] = v[e];
    }
    __syncwarp();
    const cand_t kth = row[k - 1];
    return kth ? cand_score(kth) : -CUDART_INF_F;
}

// Same result as warp_compact_row for k <= 32 and cnt <= 32, with less work: the kept list
// (one key per lane, already sorted) is merged with the sorted pending keys instead of sorting
// all slots again.  max(list[i], pending[31-i]) holds the 32 largest of both and is bitonic, so
// five more compare-exchange stages sort it.
__device__ __forceinline__ float warp_merge_row32(cand_t* row, int k, int cnt, int lane) {
    __syncwarp();
    cand_t lst = (lane < k) ? row[lane] : 0ull;
    cand_t pend[1] = {(lane < cnt) ? row[k + lane] : 0ull};
    warp_sort_desc<1>(pend, lane);
    const cand_t rev = __shfl_sync(0xFFFFFFFFu, pend[0], 31 - lane);
    cand_t m = cmax(lst, rev);
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) {
        const cand_t o = __shfl_xor_sync(0xFFFFFFFFu, m, j);
        m = ((lane & j) == 0) ? cmax(m, o) : cmin(m, o);
    }
    __syncwarp();
    if (lane < k) row[lane] = m;
    const cand_t kth = __shfl_sync(0xFFFFFFFFu, m, k - 1);
    __syncwarp();
    return kth ? cand_score(kth) : -CUDART_INF_F;
}

// Same result as warp_compact_row for k <= 32 and any cnt: the pending keys are taken 32 at a
// time, each chunk is sorted on its own (one key per lane) and merged into the kept list as in
// warp_merge_row32.  21 compare-exchange stages of one key per lane per chunk instead of
// log^2(CAP) stages of CAP/32 keys per lane over the whole buffer.
__device__ __forceinline__ float warp_merge_row_chunks(cand_t* row, int k, int cnt, int lane) {
    __syncwarp();
    cand_t m = (lane < k) ? row[lane] : 0ull;
    for (int c0 = 0; c0 < cnt; c0 += 32) {
        cand_t pend[1] = {(c0 + lane < cnt) ? row[k + c0 + lane] : 0ull};
        warp_sort_desc<1>(pend, lane);
        const cand_t rev = __shfl_sync(0xFFFFFFFFu, pend[0], 31 - lane);
        m = cmax(m, rev);
#pragma unroll
        for (int j = 16; j > 0; j >>= 1) {
            const cand_t o = __shfl_xor_sync(0xFFFFFFFFu, m, j);
            m = ((lane & j) == 0) ? cmax(m, o) : cmin(m, o);
        }
    }
    __syncwarp();
    if (lane < k) row[lane] = m;
    const cand_t kth = __shfl_sync(0xFFFFFFFFu, m, k - 1);
    __syncwarp();
    return kth ? cand_score(kth) : -CUDART_INF_F;
}

// Out-of-line entry points: compaction is rare, so one copy of its code is shared by all call
// sites and stays out of the hot loop's instruction stream.
template <int E>
__device__ __noinline__ float compact_row_outlined(cand_t* row, int k, int cnt) {
    const int lane = threadIdx.x & 31;
    if (E == 2 && k <= 32 && cnt <= 32) return warp_merge_row32(row, k, cnt, lane);
    return warp_compact_row<E>(row, k, cnt, lane);
}

// Write a finished row: slots [0,k) -> topk_idx / topk_score (empty slots: -1 / -inf).
__device__ __forceinline__ void warp_store_row(const cand_t* row, int k, int lane,
                                               int32_t* idx_out, float* score_out) {
    for (int t = lane; t < k; t += 32) {
        const cand_t c = row[t];
        idx_out[t] = c ? cand_index(c) : -1;
        score_out[t] = c ? cand_score(c) : -CUDART_INF_F;
    }
}

}  // namespace kmip
