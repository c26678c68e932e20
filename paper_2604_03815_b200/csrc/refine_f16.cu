// Rescoring kernel of the half-precision prefilter sweep (second half of Algorithm 1 line 3).
//
// score_select_f16.cu leaves, for every (query, head), the L best 8-key groups by the fp16 maximum
// of their tensor-core scores (L = k + slack).  This kernel turns them into the exact answer:
//   1. m_k = k-th largest group maximum.  The k groups at or above it each hold a key whose exact score
//      is at least lowS = m_k - err(m_k), so the true k-th best score t_k is at least lowS, and a group
//      whose maximum g satisfies g + err(g) < lowS cannot hold one of the k best keys: it is skipped.
//      err(T) = a + r |T| bounds |fp16 score - exact scaled score| (f16_filter.cuh).
//   2. The keys of the other groups are scored again - fp32 fused multiply-adds over the bf16 values in
//      index order, read from K in place - and the k best under (score desc, key asc) are kept with the
//      running top-k buffer of the CUDA-core kernel.
//   3. If the sweep's list was full, groups it dropped have maxima at most g_min, the smallest one
//      kept.  When g_min + err(g_min) reaches the k-th best exact score found, a dropped group could
//      still hold a better key: the row goes to the redo list and the exact CUDA-core kernel
//      recomputes it from all keys.  That needs more than L groups within the error bound of the
//      k-th best score, which well-separated scores never produce; rows whose keys tie massively do.
// One warp per (query, head); one candidate key per lane and step.
#include <algorithm>

#include "common.cuh"
#include "f16_filter.cuh"
#include "topk_buffer.cuh"

#include <cuda_fp16.h>

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr unsigned FULL = 0xFFFFFFFFu;

__device__ inline int graph_end_of(const int32_t* offs, int G, int N, int i) {
    if (offs == nullptr) return N;
    int a = 0, b = G;
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (__ldg(offs + m) <= i) a = m; else b = m;
    }
    return max(0, min(N, __ldg(offs + a + 1)));
}

template <int D, int E, int LIST>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
refine_f16_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                  const int32_t* __restrict__ offs, int G, int N, int H, int k,
                  const uint32_t* __restrict__ cand_word, const uint16_t* __restrict__ cand_half,
                  const F16HeadStat* __restrict__ stat, int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                  StatusBlock* __restrict__ sb, int* __restrict__ redo_list) {
    if (sb->status != KMIP_OK) return;
    using T = __nv_bfloat16;
    constexpr int CAP = 32 * E;
    constexpr int EPL = (LIST + 31) / 32;  // list entries per lane
    constexpr int KSTEPS = D / 16;
    static_assert(E <= 4 && LIST <= 64 && D <= 32, "k <= 32, head widths 16 and 32");
    __shared__ cand_t s_rows[kWarpsPerBlock][CAP];
    __shared__ float s_q[kWarpsPerBlock][D];
    __shared__ uint32_t s_words[kWarpsPerBlock][LIST];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    cand_t* row = s_rows[wib];
    float* q = s_q[wib];
    uint32_t* words = s_words[wib];
    const long long n_rows = (long long)N * H;
    const int room = CAP - k;

    for (long long r = (long long)blockIdx.x * kWarpsPerBlock + wib; r < n_rows;
         r += (long long)gridDim.x * kWarpsPerBlock) {
        const int i = (int)(r / H), h = (int)(r % H);
        const int hi = graph_end_of(offs, G, N, i);

        // the row's groups: entry t in lane t%32, register t/32
        uint32_t word[EPL];
        float g[EPL];
        bool valid[EPL];
        int n_valid = 0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const int t = e * 32 + lane;
            word[e] = 0u;
            g[e] = -CUDART_INF_F;
            valid[e] = false;
            if (t < LIST) {
                const unsigned short hb = __ldg(cand_half + (size_t)r * LIST + t);
                // empty slots: the four-pipeline sweep marks them by the half 0xFFFF and never writes their
                // group word, the ring sweep writes an all-ones word
                if (hb != 0xFFFFu) {
                    word[e] = __ldg(cand_word + (size_t)r * LIST + t);
                    valid[e] = word[e] != 0xFFFFFFFFu;
                    if (valid[e]) g[e] = __half2float(__ushort_as_half(hb));
                }
            }
            n_valid += __popc(__ballot_sync(FULL, valid[e]));
        }

        // the query row and its norms; error bound of the fp16 scores in the scaled units of the sweep
        __syncwarp();
        float qc = 0.0f;
        if (lane < D) qc = Elem<T>::load(Q + (size_t)r * D + lane);
        if (lane < D) q[lane] = qc;
        for (int t = lane; t < k; t += 32) row[t] = 0ull;
        float q2 = qc * qc, qa2 = lane < 16 ? qc * qc : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            q2 += __shfl_xor_sync(FULL, q2, o);
            qa2 += __shfl_xor_sync(FULL, qa2, o);
        }
        const F16HeadStat hs = stat[h];
        const float sq = f16_scale_from_n2max(hs.q_n2max), sk = f16_scale_from_n2max(hs.k_n2max);
        const float sc = sq * sk;  // scaled score = sc * score, a power of two
        const float nq = sqrtf(q2) * sq * 1.00001f, nqa = sqrtf(qa2) * sq * 1.00001f;
        const float nk = sqrtf(hs.k_n2max) * sk, nka = sqrtf(hs.k_first16_n2max) * sk;
        const float ea = f16_abs_err(KSTEPS, nqa, nka, nq, nk) * 1.0001f;
        const float er = kF16RelErr;
        const float fp32_err = 4e-6f * nq * nk;  // of the fp32 rescoring below, in scaled units
        __syncwarp();

        // m_k: the entry that k-1 entries beat (value desc, slot asc)
        float lowS = -CUDART_INF_F;
        float g_min = CUDART_INF_F;
#pragma unroll
        for (int e = 0; e < EPL; ++e) g_min = fminf(g_min, valid[e] ? g[e] : CUDART_INF_F);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) g_min = fminf(g_min, __shfl_xor_sync(FULL, g_min, o));
        if (n_valid >= k) {
            int rank[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) rank[e] = 0;
#pragma unroll
            for (int e2 = 0; e2 < EPL; ++e2) {
#pragma unroll 8
                for (int l = 0; l < 32; ++l) {
                    const float og = __shfl_sync(FULL, g[e2], l);
                    const int ot = e2 * 32 + l;
#pragma unroll
                    for (int e = 0; e < EPL; ++e)
                        rank[e] += (og > g[e] || (og == g[e] && ot < e * 32 + lane)) ? 1 : 0;
                }
            }
            float mk = -CUDART_INF_F;
#pragma unroll
            for (int e = 0; e < EPL; ++e)
                if (valid[e] && rank[e] == k - 1) mk = g[e];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mk = fmaxf(mk, __shfl_xor_sync(FULL, mk, o));
            lowS = mk - ea - er * fabsf(mk);
        }

        // groups that may hold one of the k best keys, compacted
        int n_kept = 0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const bool keep = valid[e] && (g[e] + ea + er * fabsf(g[e]) >= lowS);
            const unsigned m = __ballot_sync(FULL, keep);
            if (keep) words[n_kept + __popc(m & ((1u << lane) - 1u))] = word[e];
            n_kept += __popc(m);
        }
        __syncwarp();

        // every key of the answer scores at least lowS / sc exactly; keep a margin for the fp32 sums
        const float floor_tau = n_valid >= k ? (lowS - fp32_err) / sc - 1e-30f : -CUDART_INF_F;
        float tau = floor_tau;
        int cnt = 0;
        constexpr int NV = D * 2 / 16;  // 16-byte vectors per key row
        constexpr int U = 2;            // steps whose loads are issued together
        for (int t0 = 0; t0 < n_kept; t0 += U * 4) {
            int jj[U];
            bool kv[U];
            uint4 raw[U][NV];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = t0 + u * 4 + (lane >> 3);
                const uint32_t wd = t < n_kept ? words[t] : 0u;
                jj[u] = (int)(wd & 0x7FFFFFFFu) + (int)(wd >> 31) + 2 * (lane & 7);
                kv[u] = t < n_kept && jj[u] < hi && kmip_check(jj[u] >= 0 && hi <= N, sb, 101);  // checks builds: key row inside K
                if (kv[u]) {
                    const uint4* kr = reinterpret_cast<const uint4*>(K + ((size_t)jj[u] * H + h) * D);
#pragma unroll
                    for (int v = 0; v < NV; ++v) raw[u][v] = __ldg(kr + v);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float s = 0.0f;
                if (kv[u]) {
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const uint32_t wv[4] = {raw[u][v].x, raw[u][v].y, raw[u][v].z, raw[u][v].w};
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            s = fmaf(q[v * 8 + 2 * x], __uint_as_float(wv[x] << 16), s);
                            s = fmaf(q[v * 8 + 2 * x + 1], __uint_as_float(wv[x] & 0xFFFF0000u), s);
                        }
                    }
                }
                const bool pass = kv[u] && (s > tau);
                const unsigned m = __ballot_sync(FULL, pass);
                if (m) {
                    if (pass) row[k + cnt + __popc(m & ((1u << lane) - 1u))] = make_cand(s, jj[u]);
                    cnt += __popc(m);
                    if (cnt > room - 32) {
                        tau = fmaxf(floor_tau, warp_merge_row_chunks(row, k, cnt, lane));
                        cnt = 0;
                    }
                }
            }
        }
        const float kth = warp_merge_row_chunks(row, k, cnt, lane);
        // a dropped group scores at most g_min + err(g_min) exactly (scaled); it matters if that reaches the
        // k-th best score found
        if (n_valid == LIST && g_min + ea + er * fabsf(g_min) >= kth * sc - fp32_err) {
            if (lane == 0) {
                const int pos = atomicAdd(&sb->n_redo, 1);
                if (kmip_check(pos >= 0 && pos < n_rows, sb, 102)) redo_list[pos] = (int)r;  // checks builds: inside the list
            }
        }
        warp_store_row(row, k, lane, topk_idx + (size_t)r * k, topk_score + (size_t)r * k);
    }
}

template <int D>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w) {
    const long long n_rows = (long long)a.N * a.H;
    const int blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
#define KMIP_LAUNCH_REFINE16(E_, LIST_) \
    refine_f16_kernel<D, E_, LIST_><<<blocks, kWarpsPerBlock * 32, 0, a.stream>>>( \
        static_cast<const __nv_bfloat16*>(a.Q), static_cast<const __nv_bfloat16*>(a.K), a.graph_offsets, a.G, (int)a.N, \
        a.H, a.k, reinterpret_cast<const uint32_t*>(a.ws + w.cand_word_off), \
        reinterpret_cast<const uint16_t*>(a.ws + w.cand_half_off), reinterpret_cast<const F16HeadStat*>(a.ws + w.f16stat_off), \
        a.topk_idx, a.topk_score, reinterpret_cast<StatusBlock*>(a.ws), reinterpret_cast<int*>(a.ws + w.redo_off))
    // the list sizes are those of score_select_f16_list
    if (a.k <= 8) KMIP_LAUNCH_REFINE16(2, 16);
    else if (a.k <= 16) KMIP_LAUNCH_REFINE16(2, 24);
    else KMIP_LAUNCH_REFINE16(4, 48);
#undef KMIP_LAUNCH_REFINE16
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_refine_f16(const FwdArgs& a, const FwdWorkspace& w) {
    return a.d == 16 ? launch_d<16>(a, w) : launch_d<32>(a, w);
}

}  // namespace kmip
