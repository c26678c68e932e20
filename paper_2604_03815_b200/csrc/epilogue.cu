// Softmax over the k kept scores fused with the gather-V weighted sum (Algorithm 1 lines 4-6).
// One warp per (query, head) row; the N x k x d tensor V_topk of line 4 is never materialised.
#include <algorithm>

#include "common.cuh"
#include "rowops.cuh"

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;

template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
softmax_gather_kernel(const T* __restrict__ V, const int32_t* __restrict__ topk_idx,
                      const float* __restrict__ topk_score, int N, int H, int k, float scale,
                      float drop_p, unsigned long long seed, T* __restrict__ out,
                      const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;  // an earlier stage failed: topk_idx was not written
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    const int lane = threadIdx.x & 31;
    const long long n_rows = (long long)N * H;
    for (long long r = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); r < n_rows;
         r += (long long)gridDim.x * kWarpsPerBlock) {
        const int h = (int)(r % H);
        int j[kMaxEntriesPerLane];
        float p[kMaxEntriesPerLane];
        load_row_softmax(topk_idx + (size_t)r * k, topk_score + (size_t)r * k, k, N, scale, lane, j, p);
        if (drop_p > 0.0f) {  // training only: the weights go through dropout before the weighted sum
            float f[kMaxEntriesPerLane];
            dropout_factors(r, k, lane, drop_p, seed, f);
#pragma unroll
            for (int e = 0; e < kMaxEntriesPerLane; ++e) p[e] *= f[e];
        }
        float acc[VEC];
        gather_weighted_sum<T, D>(V, H, h, k, lane, j, p, acc);
        if (lane < LPR) Elem<T>::store_vec(out + (size_t)r * D + lane * VEC, acc);
    }
}

template <typename T, int D>
cudaError_t launch_d(const FwdArgs& a) {
    const long long n_rows = (long long)a.N * a.H;
    const int blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
    softmax_gather_kernel<T, D><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>(
        static_cast<const T*>(a.V), a.topk_idx, a.topk_score, (int)a.N, a.H, a.k,
        1.0f / sqrtf((float)a.d), a.drop_p, a.seed, static_cast<T*>(a.out), reinterpret_cast<const StatusBlock*>(a.ws));
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(const FwdArgs& a) {
    switch (a.d) {
        case 16: return launch_d<T, 16>(a);
        case 32: return launch_d<T, 32>(a);
        case 64: return launch_d<T, 64>(a);
        case 128: return launch_d<T, 128>(a);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_softmax_gather(const FwdArgs& a) {
    return a.mode == KMIP_FP32_EXACT ? launch_t<float>(a) : launch_t<__nv_bfloat16>(a);
}

}  // namespace kmip
