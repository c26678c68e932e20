// CUDA-core score + running top-k kernel (Algorithm 1 lines 2-3), one warp per (query, head).
//
// This is the KMIP_FP32_EXACT path: every score is d fused multiply-adds in fp32, in index
// order c = 0..d-1.  It also serves bf16 storage for (d, k) combinations the tensor-core
// kernel does not cover.  The N x N score matrix is never stored: each lane scores one key
// per step and the warp appends the survivors of the threshold test to the row's buffer.
#include <algorithm>

#include "common.cuh"
#include "topk_buffer.cuh"

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;

// Graph range of row i: binary search for the last offset <= i, skipping empty graphs.
__device__ inline void graph_range(const int32_t* offs, int G, int N, int i, int& lo, int& hi) {
    if (offs == nullptr) { lo = 0; hi = N; return; }
    int a = 0, b = G;  // invariant: offs[a] <= i, answer in [a, b)
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (__ldg(offs + m) <= i) a = m; else b = m;
    }
    lo = max(0, min(N, __ldg(offs + a)));
    hi = max(lo, min(N, __ldg(offs + a + 1)));
}

template <typename T, int D, int E>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
score_select_exact_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                          const int32_t* __restrict__ offs, int G, int N, int H, int k,
                          int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                          const StatusBlock* __restrict__ sb, const int* __restrict__ redo_list) {
    if (sb->status != KMIP_OK) return;  // the plan kernel rejected the offsets
    constexpr int CAP = 32 * E;
    constexpr int VEC = Elem<T>::kVec;
    __shared__ cand_t s_rows[kWarpsPerBlock][CAP];
    __shared__ float s_q[kWarpsPerBlock][D];

    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    cand_t* row = s_rows[wib];
    float* q = s_q[wib];
    // redo_list: only the (row, head) pairs the rescoring kernel of the half-precision prefilter listed
    const long long n_rows = redo_list ? (long long)sb->n_redo : (long long)N * H;
    const int room = CAP - k;  // pending slots

    for (long long x = (long long)blockIdx.x * kWarpsPerBlock + wib; x < n_rows;
         x += (long long)gridDim.x * kWarpsPerBlock) {
        const long long r = redo_list ? (long long)__ldg(redo_list + x) : x;
        const int i = (int)(r / H), h = (int)(r % H);
        int lo, hi;
        graph_range(offs, G, N, i, lo, hi);

        __syncwarp();
        for (int c = lane; c < D; c += 32) q[c] = Elem<T>::load(Q + ((size_t)i * H + h) * D + c);
        for (int t = lane; t < k; t += 32) row[t] = 0ull;
        __syncwarp();

        float tau = -CUDART_INF_F;
        int cnt = 0;
        for (int j0 = lo; j0 < hi; j0 += 32) {
            const int j = j0 + lane;
            const bool valid = j < hi;
            float s = 0.0f;
            if (valid) {
                const T* kr = K + ((size_t)j * H + h) * D;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += VEC) {
                    float kv[VEC];
                    Elem<T>::load_vec(kr + c0, kv);
#pragma unroll
                    for (int c = 0; c < VEC; ++c) s = fmaf(q[c0 + c], kv[c], s);
                }
            }
            const bool pass = valid && (s > tau);
            const unsigned m = __ballot_sync(0xFFFFFFFFu, pass);
            if (m) {
                if (pass) row[k + cnt + __popc(m & ((1u << lane) - 1u))] = make_cand(s, j);
                cnt += __popc(m);
                if (cnt > room - 32) {
                    tau = warp_compact_row<E>(row, k, cnt, lane);
                    cnt = 0;
                }
            }
        }
        warp_compact_row<E>(row, k, cnt, lane);
        warp_store_row(row, k, lane, topk_idx + (size_t)r * k, topk_score + (size_t)r * k);
    }
}

template <typename T, int D>
cudaError_t launch_d(const FwdArgs& a, const int* redo_list = nullptr) {
    const long long n_rows = (long long)a.N * a.H;
    // the redo pass does not know its row count on the host: a grid that covers a few thousand rows at once
    const int blocks = redo_list ? sm_count() * 4
                                 : (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 64);
    const T* Q = static_cast<const T*>(a.Q);
    const T* K = static_cast<const T*>(a.K);
    const dim3 grid(blocks), block(kWarpsPerBlock * 32);
    // pending room CAP-k must hold one 32-key step beyond the compaction trigger
#define KMIP_LAUNCH_EXACT(E_) \
    score_select_exact_kernel<T, D, E_><<<grid, block, 0, a.stream>>>( \
        Q, K, a.graph_offsets, a.G, (int)a.N, a.H, a.k, a.topk_idx, a.topk_score, \
        reinterpret_cast<const StatusBlock*>(a.ws), redo_list)
    if (a.k <= 16) KMIP_LAUNCH_EXACT(2);
    else if (a.k <= 96) KMIP_LAUNCH_EXACT(4);
    else KMIP_LAUNCH_EXACT(8);
#undef KMIP_LAUNCH_EXACT
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

cudaError_t launch_score_select_exact(const FwdArgs& a) {
    return a.mode == KMIP_FP32_EXACT ? launch_t<float>(a) : launch_t<__nv_bfloat16>(a);
}

// The rows the half-precision prefilter could not decide (bf16 storage, head widths 16 and 32), again
// from all keys of their graph; overwrites their topk_idx / topk_score.
cudaError_t launch_score_select_exact_redo(const FwdArgs& a, const FwdWorkspace& w) {
    const int* redo = reinterpret_cast<const int*>(a.ws + w.redo_off);
    return a.d == 16 ? launch_d<__nv_bfloat16, 16>(a, redo) : launch_d<__nv_bfloat16, 32>(a, redo);
}

}  // namespace kmip
