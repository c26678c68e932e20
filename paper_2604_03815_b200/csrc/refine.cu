// Rescoring kernel of the tensor-core path (second half of Algorithm 1 line 3).
//
// The sweep kernel leaves, for every (query, head), the k best 8-key groups: topk_idx holds each
// group's first key, topk_score its maximum (tensor-core score).  Those groups contain the k best
// keys, so this kernel scores the 8k keys of a row again - fp32 fused multiply-adds over the
// bf16 values, in index order - keeps the k best under (score desc, key asc) with the same
// running top-k buffer as the CUDA-core kernel, and overwrites topk_idx / topk_score with them.
// One warp per (query, head); one candidate key per lane and step.
#include <algorithm>

#include "common.cuh"
#include "topk_buffer.cuh"

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kGroup = 8;  // keys per group, fixed by the sweep kernel

__device__ inline int graph_end(const int32_t* offs, int G, int N, int i) {
    if (offs == nullptr) return N;
    int a = 0, b = G;
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (__ldg(offs + m) <= i) a = m; else b = m;
    }
    return max(0, min(N, __ldg(offs + a + 1)));
}

// REGROUPED: `Kp` is the bf16 copy of K regrouped by head, [H, N, D] (tensor-core mode); otherwise it is
// K itself, [N, H, D] (fp32 mode, scores by fp32 FMA in index order as in the exact kernel).
template <typename T, int D, int E, bool REGROUPED>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
refine_topk_kernel(const T* __restrict__ Q, const T* __restrict__ Kp, const int32_t* __restrict__ offs, int G,
                   int N, int H, int k, int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                   const StatusBlock* __restrict__ sb, const int* __restrict__ kperm) {
    if (sb->status != KMIP_OK) return;
    constexpr int CAP = 32 * E;
    static_assert((sizeof(T) == 2) == REGROUPED, "bf16 keys come regrouped, fp32 keys in place");
    __shared__ cand_t s_rows[kWarpsPerBlock][CAP];
    __shared__ float s_q[kWarpsPerBlock][D];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    cand_t* row = s_rows[wib];
    float* q = s_q[wib];
    const long long n_rows = (long long)N * H;
    const int room = CAP - k;

    for (long long r = (long long)blockIdx.x * kWarpsPerBlock + wib; r < n_rows;
         r += (long long)gridDim.x * kWarpsPerBlock) {
        const int i = (int)(r / H), h = (int)(r % H);
        const int hi = graph_end(offs, G, N, i);

        // the row's groups: entry t in lane t%32, register t/32
        int gid[4];
        float theta = CUDART_INF_F;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int t = e * 32 + lane;
            gid[e] = -1;
            if (t < k) {
                gid[e] = topk_idx[(size_t)r * k + t];
                const float gmax = topk_score[(size_t)r * k + t];
                theta = fminf(theta, gid[e] >= 0 ? gmax : -CUDART_INF_F);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) theta = fminf(theta, __shfl_xor_sync(0xFFFFFFFFu, theta, o));
        // every key of the answer scores at least theta (the k-th best group maximum) up to the
        // difference between tensor-core and fp32 accumulation; keep a margin for that
        const float floor_tau = theta - 1e-4f * fabsf(theta) - 1e-30f;

        __syncwarp();
        for (int c = lane; c < D; c += 32) q[c] = Elem<T>::load(Q + ((size_t)i * H + h) * D + c);
        for (int t = lane; t < k; t += 32) row[t] = 0ull;
        __syncwarp();

        // Two attempts at most.  The margin above is relative to theta, so when the k-th best group maximum
        // lies within rounding of zero the fp32 sums below can fall short of it by more than the margin and a
        // key of the answer would be dropped; the row then comes out with fewer than k keys although its
        // groups hold more, and it is scanned again without a floor.
        for (int attempt = 0; attempt < 2; ++attempt) {
        const float floor_now = attempt == 0 ? floor_tau : -CUDART_INF_F;
        int n_seen = 0;  // keys of the row's groups that exist (inside the graph)
        float tau = floor_now;
        int cnt = 0;
        constexpr int GPR = 32 / kGroup;           // groups scored per step (one key per lane)
        constexpr int NV = D * (int)sizeof(T) / 16;  // 16-byte vectors per key row
        constexpr int U = (NV <= 8) ? 2 : 1;       // steps whose loads are issued together
        for (int t0 = 0; t0 < k; t0 += U * GPR) {
            int jj[U];
            bool valid[U];
            uint4 raw[U][NV];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int tb = t0 + u * GPR, t = tb + lane / kGroup;
                int g = -1;
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (e == (tb >> 5)) g = __shfl_sync(0xFFFFFFFFu, gid[e], t & 31);
                jj[u] = g + (lane % kGroup);
                valid[u] = t < k && g >= 0 && jj[u] < hi &&
                           kmip_check(jj[u] >= 0 && hi <= N, const_cast<StatusBlock*>(sb), 101);  // checks builds: key row inside K
                if (valid[u]) {
                    // regrouped by head, the 8 keys of a group are 8 consecutive rows
                    const uint4* kr = reinterpret_cast<const uint4*>(
                        REGROUPED ? Kp + ((size_t)h * N + jj[u]) * D : Kp + ((size_t)jj[u] * H + h) * D);
#pragma unroll
                    for (int v = 0; v < NV; ++v) raw[u][v] = __ldg(kr + v);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float s = 0.0f;
                if (valid[u]) {
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const uint32_t wv[4] = {raw[u][v].x, raw[u][v].y, raw[u][v].z, raw[u][v].w};
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            if constexpr (sizeof(T) == 2) {
                                s = fmaf(q[v * 8 + 2 * x], __uint_as_float(wv[x] << 16), s);
                                s = fmaf(q[v * 8 + 2 * x + 1], __uint_as_float(wv[x] & 0xFFFF0000u), s);
                            } else {
                                s = fmaf(q[v * 4 + x], __uint_as_float(wv[x]), s);
                            }
                        }
                    }
                }
                n_seen += __popc(__ballot_sync(0xFFFFFFFFu, valid[u]));
                const bool pass = valid[u] && (s > tau);
                const unsigned m = __ballot_sync(0xFFFFFFFFu, pass);
                if (m) {
                    // pruned sweep: the groups are positions of the sweep's key order; the answer names the keys
                    if (pass) row[k + cnt + __popc(m & ((1u << lane) - 1u))] = make_cand(s, kperm ? __ldg(kperm + jj[u]) : jj[u]);
                    cnt += __popc(m);
                    if (cnt > room - 32) {
                        tau = fmaxf(floor_now, E <= 4 ? warp_merge_row_chunks(row, k, cnt, lane) : warp_compact_row<E>(row, k, cnt, lane));
                        cnt = 0;
                    }
                }
            }
        }
        // E <= 4 serves k <= 32: one kept key per lane, so the pending keys can be merged in 32-key chunks
        if (E <= 4) warp_merge_row_chunks(row, k, cnt, lane); else warp_compact_row<E>(row, k, cnt, lane);
        __syncwarp();
        const int n_kept = __popc(__ballot_sync(0xFFFFFFFFu, lane < k && row[lane] != 0ull)) +
                           ((k > 32) ? __popc(__ballot_sync(0xFFFFFFFFu, lane + 32 < k && row[lane + 32] != 0ull)) +
                                       __popc(__ballot_sync(0xFFFFFFFFu, lane + 64 < k && row[lane + 64] != 0ull)) +
                                       __popc(__ballot_sync(0xFFFFFFFFu, lane + 96 < k && row[lane + 96] != 0ull)) : 0);
        if (n_kept >= min(k, n_seen)) break;
        __syncwarp();
        for (int t = lane; t < k; t += 32) row[t] = 0ull;
        __syncwarp();
        }
        warp_store_row(row, k, lane, topk_idx + (size_t)r * k, topk_score + (size_t)r * k);
    }
}

template <typename T, int D>
cudaError_t launch_d(const FwdArgs& a, const T* keys, const int* kperm = nullptr) {
    constexpr bool REGROUPED = sizeof(T) == 2;
    const long long n_rows = (long long)a.N * a.H;
    const int blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
#define KMIP_LAUNCH_REFINE(E_) \
    refine_topk_kernel<T, D, E_, REGROUPED><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>( \
        static_cast<const T*>(a.Q), keys, a.graph_offsets, a.G, (int)a.N, a.H, a.k, \
        a.topk_idx, a.topk_score, reinterpret_cast<const StatusBlock*>(a.ws), kperm)
    // pending room CAP-k: the survivors of a row (rarely more than 2k) should fit without intermediate
    // compactions, and the final sort costs log^2(CAP) compare-exchange stages
    if (a.k <= 16) KMIP_LAUNCH_REFINE(2);
    else if (a.k <= 32) KMIP_LAUNCH_REFINE(4);
    else KMIP_LAUNCH_REFINE(8);
#undef KMIP_LAUNCH_REFINE
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_refine_topk(const FwdArgs& a, const FwdWorkspace& w) {
    using T = __nv_bfloat16;
    const T* keys = reinterpret_cast<const T*>(a.ws + w.kpack_off);
    const int* kperm = w.prune ? reinterpret_cast<const int*>(a.ws + w.kperm_off) : nullptr;
    switch (a.d) {
        case 16: return launch_d<T, 16>(a, keys, kperm);
        case 32: return launch_d<T, 32>(a, keys, kperm);
        case 64: return launch_d<T, 64>(a, keys, kperm);
        case 128: return launch_d<T, 128>(a, keys, kperm);
        default: return cudaErrorInvalidValue;
    }
}

// fp32 mode (tiled CUDA-core sweep): the keys are read in place.
cudaError_t launch_refine_topk_fp32(const FwdArgs& a) {
    const float* keys = static_cast<const float*>(a.K);
    switch (a.d) {
        case 16: return launch_d<float, 16>(a, keys);
        case 32: return launch_d<float, 32>(a, keys);
        case 64: return launch_d<float, 64>(a, keys);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace kmip
