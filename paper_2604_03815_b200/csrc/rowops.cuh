// Warp-level building blocks for the gather stages (Algorithm 1 lines 4-6 and their backward):
// softmax over the k kept scores of one (query, head) row, and the weighted sum of gathered rows
// with 16-byte vector loads.
#pragma once

#include "common.cuh"
#include <math_constants.h>

namespace kmip {

constexpr int kMaxEntriesPerLane = 4;  // k <= 128

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Entry t of a row lives in lane t%32, register t/32.  Loads the row's indices and scores and
// turns the scores into softmax weights p_t = exp((s_t - max)/sqrt(d)) / sum (Algorithm 1 line 5).
// Empty slots (index < 0) and indices outside [0, N) get weight 0.
__device__ __forceinline__ void load_row_softmax(const int32_t* idx_row, const float* score_row, int k, int N,
                                                 float scale, int lane,
                                                 int (&j)[kMaxEntriesPerLane], float (&p)[kMaxEntriesPerLane]) {
    float m = -CUDART_INF_F;
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) {
        const int t = e * 32 + lane;
        j[e] = -1;
        p[e] = -CUDART_INF_F;
        if (t < k) {
            j[e] = __ldg(idx_row + t);
            if (j[e] >= N) j[e] = -1;  // never follow an index outside the batch
            const float s = __ldg(score_row + t);
            if (j[e] >= 0) p[e] = s;
        }
        m = fmaxf(m, p[e]);
    }
    m = warp_max(m);
    float z = 0.0f;
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) {
        p[e] = (j[e] >= 0) ? __expf((p[e] - m) * scale) : 0.0f;
        z += p[e];
    }
    z = warp_sum(z);
    const float inv = z > 0.0f ? 1.0f / z : 0.0f;
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) p[e] *= inv;
}

// Attention dropout on the k weights of row r (= query * H + head): factor 1/(1-drop) when the slot's
// counter-based uniform is >= drop, else 0.  The draw of slot t is the (r*k + t + 1)-th SplitMix64
// output for `seed`, top 24 bits / 2^24.  f[e] belongs to entry t = e*32 + lane.
__device__ __forceinline__ void dropout_factors(long long r, int k, int lane, float drop, unsigned long long seed,
                                                float (&f)[kMaxEntriesPerLane]) {
    const float keep_scale = 1.0f / (1.0f - drop);
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) {
        const unsigned long long pair = (unsigned long long)r * (unsigned long long)k + (unsigned long long)(e * 32 + lane);
        unsigned long long z = seed + (pair + 1ull) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z = z ^ (z >> 31);
        const float u = (float)(unsigned)(z >> 40) * (1.0f / 16777216.0f);  // 24 bits: exact in fp32
        f[e] = (u >= drop) ? keep_scale : 0.0f;
    }
}

// acc (per lane: VEC columns of the part this lane owns) = sum_t w_t * X[j_t, h, part*VEC ..].
// LPR = D/VEC lanes share one gathered row (one 16-byte load each), 32/LPR rows per round.
// After the call lanes 0..LPR-1 hold the full sums for their part.
template <typename T, int D>
__device__ __forceinline__ void gather_weighted_sum(const T* __restrict__ X, int H, int h, int k, int lane,
                                                    const int (&j)[kMaxEntriesPerLane],
                                                    const float (&w)[kMaxEntriesPerLane],
                                                    float (&acc)[Elem<T>::kVec]) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int EPW = 32 / LPR;
    static_assert(LPR >= 1 && LPR <= 32, "row width");
    const int part = lane % LPR, sub = lane / LPR;
#pragma unroll
    for (int c = 0; c < VEC; ++c) acc[c] = 0.0f;
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) {
        if (e * 32 < k) {
#pragma unroll
            for (int base = 0; base < 32; base += EPW) {
                if (e * 32 + base >= k) break;
                const int src = base + sub;
                const int jj = __shfl_sync(0xFFFFFFFFu, j[e], src);
                const float ww = __shfl_sync(0xFFFFFFFFu, w[e], src);
                if (jj >= 0) {
                    float v[VEC];
                    Elem<T>::load_vec(X + ((size_t)jj * H + h) * D + part * VEC, v);
#pragma unroll
                    for (int c = 0; c < VEC; ++c) acc[c] = fmaf(ww, v[c], acc[c]);
                }
            }
        }
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int c = 0; c < VEC; ++c) acc[c] += __shfl_xor_sync(0xFFFFFFFFu, acc[c], o);
    }
}

// dots[e] of lane l = g . X[j[e] of lane l, h, :] for the row's entries (entry t in lane t % 32, register t / 32), with
// the same lane layout as gather_weighted_sum: LPR lanes share one gathered row, one 16-byte load each, so a load
// instruction touches 32 / LPR rows instead of 32; the partial sums of a row are added across its lanes and handed
// to the entry's own lane.  g is the row-major vector of D elements at `g_row`.
template <typename T, int D>
__device__ __forceinline__ void gather_dot(const T* __restrict__ X, int H, int h, int k, int lane, const T* __restrict__ g_row,
                                           const int (&j)[kMaxEntriesPerLane], float (&dots)[kMaxEntriesPerLane]) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int EPW = 32 / LPR;
    const int part = lane % LPR, sub = lane / LPR;
    float gv[VEC];
    Elem<T>::load_vec(g_row + part * VEC, gv);
#pragma unroll
    for (int e = 0; e < kMaxEntriesPerLane; ++e) {
        dots[e] = 0.0f;
        if (e * 32 < k) {
#pragma unroll
            for (int base = 0; base < 32; base += EPW) {
                if (e * 32 + base >= k) break;
                const int jj = __shfl_sync(0xFFFFFFFFu, j[e], base + sub);
                float s = 0.0f;
                if (jj >= 0) {
                    float v[VEC];
                    Elem<T>::load_vec(X + ((size_t)jj * H + h) * D + part * VEC, v);
#pragma unroll
                    for (int c = 0; c < VEC; ++c) s = fmaf(gv[c], v[c], s);
                }
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
                // the entry of lane l was gathered by the lanes (l % EPW) * LPR ... in the round base = l - l % EPW
                const float t = __shfl_sync(0xFFFFFFFFu, s, (lane % EPW) * LPR);
                if (lane - lane % EPW == base) dots[e] = t;
            }
        }
    }
}

}  // namespace kmip
