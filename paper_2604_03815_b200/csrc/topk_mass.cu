// Diagnostic of the paper's App. I ("cumulative attention weight"): the share of the FULL softmax
// over all keys of the query's graph that falls on the k keys the forward pass kept,
//   mass[i,h] = sum_t exp(s_t / sqrt(d)) / sum_j exp(q_i . k_j / sqrt(d)),   s = topk_score[i,h,:].
// The denominator needs every score of the row again; they are computed on CUDA cores in fp32
// (one thread per query row, keys staged in shared memory as in score_select_fp32.cu) and folded
// into a running log-sum-exp eight keys at a time, so nothing of size N x N is stored here either.
#include <algorithm>

#include "common.cuh"
#include <math_constants.h>

namespace kmip {

namespace {

constexpr int ROWS = 128;  // query rows per block = threads per block
constexpr int TK = 64;     // keys per shared-memory tile
constexpr int GK = 8;      // keys folded into the running sum at a time

template <typename T, int D>
__global__ void __launch_bounds__(ROWS)
topk_mass_kernel(const T* __restrict__ Q, const T* __restrict__ K, const WorkItem* __restrict__ items,
                 const StatusBlock* __restrict__ sb, int H, int k, const float* __restrict__ topk_score,
                 float* __restrict__ mass) {
    if (sb->status != KMIP_OK) return;  // the plan kernel rejected the offsets
    constexpr int VEC = Elem<T>::kVec;
    __shared__ __align__(16) float sK[TK * D];
    const int tid = threadIdx.x;
    const float scale2 = 1.4426950408889634f / sqrtf((float)D);  // log2(e) / sqrt(d): exponentials in base 2
    const int n_items = sb->n_items;
    const long long total = (long long)n_items * H;
    for (long long w = blockIdx.x; w < total; w += gridDim.x) {
        const int h = (int)(w / n_items);
        const WorkItem it = items[w % n_items];
        const bool rvalid = tid < it.nrows;
        const int row = it.row0 + (rvalid ? tid : 0);
        float q[D];
#pragma unroll
        for (int c = 0; c < D; c += VEC) {
            float t[VEC];
            Elem<T>::load_vec(Q + ((size_t)row * H + h) * D + c, t);
#pragma unroll
            for (int x = 0; x < VEC; ++x) q[c + x] = t[x] * scale2;
        }
        float m = -CUDART_INF_F, z = 0.0f;  // running maximum and sum of 2^(s - m)
        for (int key0 = it.key_lo; key0 < it.key_hi; key0 += TK) {
            const int nvalid = min(TK, it.key_hi - key0);
            __syncthreads();  // everybody is done with the previous tile
            for (int x = tid; x < nvalid * (D / VEC); x += ROWS) {
                const int r = x / (D / VEC), v = x % (D / VEC);
                float t[VEC];
                Elem<T>::load_vec(K + ((size_t)(key0 + r) * H + h) * D + v * VEC, t);
#pragma unroll
                for (int y = 0; y < VEC; ++y) sK[r * D + v * VEC + y] = t[y];
            }
            __syncthreads();
#pragma unroll 1
            for (int g = 0; g * GK < nvalid; ++g) {
                float acc[GK];
#pragma unroll
                for (int j = 0; j < GK; ++j) acc[j] = 0.0f;
                const float* kg = sK + g * GK * D;
#pragma unroll
                for (int c = 0; c < D; c += 4) {
#pragma unroll
                    for (int j = 0; j < GK; ++j) {
                        const float4 kv = *reinterpret_cast<const float4*>(kg + j * D + c);  // same address in every thread
                        acc[j] = fmaf(q[c], kv.x, acc[j]);
                        acc[j] = fmaf(q[c + 1], kv.y, acc[j]);
                        acc[j] = fmaf(q[c + 2], kv.z, acc[j]);
                        acc[j] = fmaf(q[c + 3], kv.w, acc[j]);
                    }
                }
                float gm = -CUDART_INF_F;
#pragma unroll
                for (int j = 0; j < GK; ++j) {
                    if (g * GK + j >= nvalid) acc[j] = -CUDART_INF_F;  // keys past the end of the graph
                    gm = fmaxf(gm, acc[j]);
                }
                const float m_new = fmaxf(m, gm);  // finite: the group holds at least one key
                float add = 0.0f;
#pragma unroll
                for (int j = 0; j < GK; ++j) add += exp2f(acc[j] - m_new);
                z = z * exp2f(m - m_new) + add;
                m = m_new;
            }
        }
        if (rvalid) {
            const float* s = topk_score + ((size_t)row * H + h) * k;
            const float sc = 1.4426950408889634f / sqrtf((float)D);
            float top = 0.0f;
            for (int t = 0; t < k; ++t) {
                const float v = __ldg(s + t);
                if (v > -CUDART_INF_F) top += exp2f(v * sc - m);
            }
            mass[(size_t)row * H + h] = z > 0.0f ? fminf(top / z, 1.0f) : 0.0f;
        }
    }
}

template <typename T, int D>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w, float* mass) {
    const long long total = (long long)w.max_items * a.H;
    const int grid = (int)std::min<long long>(total, (long long)sm_count() * 16);
    topk_mass_kernel<T, D><<<grid, ROWS, 0, a.stream>>>(
        static_cast<const T*>(a.Q), static_cast<const T*>(a.K), reinterpret_cast<const WorkItem*>(a.ws + w.items_off),
        reinterpret_cast<const StatusBlock*>(a.ws), a.H, a.k, a.topk_score, mass);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(const FwdArgs& a, const FwdWorkspace& w, float* mass) {
    switch (a.d) {
        case 16: return launch_d<T, 16>(a, w, mass);
        case 32: return launch_d<T, 32>(a, w, mass);
        case 64: return launch_d<T, 64>(a, w, mass);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

// Work items of 128 rows must be in the workspace (launch_plan with rows_per_item = 128).
cudaError_t launch_topk_mass(const FwdArgs& a, const FwdWorkspace& w, float* mass) {
    return a.mode == KMIP_FP32_EXACT ? launch_t<float>(a, w, mass) : launch_t<__nv_bfloat16>(a, w, mass);
}

}  // namespace kmip
