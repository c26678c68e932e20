// Rescoring kernel of the half-precision prefilter sweep (second half of Algorithm 1 line 3).
//
// score_select_f16.cu leaves, for every (query, head), the L best 8-key groups by the fp16 maximum
// of their tensor-core scores (L = k + slack).  This kernel turns them into the exact answer:
//   1. m_k = k-th largest group maximum (a 16-step search over the bits of the half-precision value).  The k groups at or above it each hold a key whose exact score
//      is at least lowS = m_k - err(m_k), so the true k-th best score t_k is at least lowS, and a group
//      whose maximum g satisfies g + err(g) < lowS cannot hold one of the k best keys: it is skipped.
//      err(T) = a + r |T| bounds |fp16 score - exact scaled score| (f16_filter.cuh).
//   2. The keys of the other groups are scored again - fp32 fused multiply-adds over the bf16 values in
//      index order (the mixed-precision instruction: exact product, one rounding, the same bits as convert +
//      fmaf), read from K in place - and the k best under (score desc, key asc) are kept with the
//      running top-k buffer of the CUDA-core kernel.
//   3. If the sweep's list was full, groups it dropped have maxima at most g_min, the smallest one
//      kept.  When g_min + err(g_min) reaches the k-th best exact score found, a dropped group could
//      still hold a better key: the row goes to the redo list and the exact CUDA-core kernel
//      recomputes it from all keys.  That needs more than L groups within the error bound of the
//      k-th best score, which well-separated scores never produce; rows whose keys tie massively do.
// One warp per (query, head); a candidate key's row is read by D / 8 neighbouring lanes.
#include <algorithm>

#include "common.cuh"
#include "f16_filter.cuh"
#include "ptx.cuh"
#include "topk_buffer.cuh"

#include <cuda_fp16.h>

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr unsigned FULL = 0xFFFFFFFFu;

// End of the graph that holds node i.  Batches of up to kOffsCached - 1 graphs search a copy of the offsets in
// shared memory: seven dependent global loads per row would otherwise be the longest chain of a small-graph batch.
constexpr int kOffsCached = 1024;
__device__ inline int graph_end_of(const int32_t* offs, const int* s_offs, int G, int N, int i) {
    if (offs == nullptr) return N;
    int a = 0, b = G;
    if (G < kOffsCached) {
        while (b - a > 1) {
            const int m = (a + b) >> 1;
            if (s_offs[m] <= i) a = m; else b = m;
        }
        return max(0, min(N, s_offs[a + 1]));
    }
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (__ldg(offs + m) <= i) a = m; else b = m;
    }
    return max(0, min(N, __ldg(offs + a + 1)));
}

// fp16 bits -> 16-bit key whose unsigned order is the order of the values (no NaNs reach this point)
__device__ __forceinline__ unsigned f16_ordered(unsigned hb) { return (hb & 0x8000u) ? (~hb & 0xFFFFu) : (hb | 0x8000u); }
__device__ __forceinline__ unsigned f16_unordered(unsigned ok) { return (ok & 0x8000u) ? (ok & 0x7FFFu) : (~ok & 0xFFFFu); }

template <int D, int E, int LIST>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, 4)
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
    __shared__ __align__(16) unsigned short s_qb[kWarpsPerBlock][D];  // the query row, bf16 bits
    __shared__ uint32_t s_words[kWarpsPerBlock][LIST];
    __shared__ int s_offs[kOffsCached];
    if (offs != nullptr && G < kOffsCached) {
        for (int x = threadIdx.x; x <= G; x += blockDim.x) s_offs[x] = __ldg(offs + x);
        __syncthreads();
    }
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    cand_t* row = s_rows[wib];
    uint32_t* words = s_words[wib];
    const long long n_rows = (long long)N * H;
    const long long stride = (long long)gridDim.x * kWarpsPerBlock;
    const int room = CAP - k;
    constexpr int P = D / 8;                   // 16-byte pieces of a key row
    constexpr int kRowStride = D * 2 + 16;     // padded: a lane per row reads 16-byte pieces without bank conflicts
    constexpr int kStageBytes = 32 * kRowStride;
    extern __shared__ __align__(16) unsigned char s_stage[];  // [warp][2 stages][32 rows]
    unsigned char* stage = s_stage + wib * 2 * kStageBytes;
    const int pl = lane % P;
    const unsigned row_bytes = (unsigned)(H * D * (int)sizeof(T));

    // a row's list (entry t in lane t % 32, register t / 32) and query element are fetched one row ahead
    uint32_t nx_word[EPL];
    unsigned nx_half[EPL];
    float nx_q = 0.0f;
    auto fetch = [&](long long r) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const int t = e * 32 + lane;
            nx_half[e] = 0xFFFFu;
            nx_word[e] = 0xFFFFFFFFu;
            if (r < n_rows && t < LIST) {
                nx_half[e] = __ldg(cand_half + (size_t)r * LIST + t);
                nx_word[e] = __ldg(cand_word + (size_t)r * LIST + t);  // never written for an empty slot: ignored below
            }
        }
        nx_q = (r < n_rows && lane < D) ? Elem<T>::load(Q + (size_t)r * D + lane) : 0.0f;
    };
    long long r = (long long)blockIdx.x * kWarpsPerBlock + wib;
    fetch(r);

    for (; r < n_rows; r += stride) {
        const int i = (int)(r / H), h = (int)(r % H);
        const int hi = graph_end_of(offs, s_offs, G, N, i);

        // empty slots: the four-pipeline sweep marks them by the half 0xFFFF and never writes their group word,
        // the ring sweep writes an all-ones word
        uint32_t word[EPL];
        unsigned okey[EPL];  // ordered 16-bit key of the group maximum; 0 for an empty slot (below every value)
        int n_valid = 0;
        unsigned ok_min = 0xFFFFu;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            word[e] = nx_word[e];
            const bool valid = nx_half[e] != 0xFFFFu && word[e] != 0xFFFFFFFFu;
            okey[e] = valid ? f16_ordered(nx_half[e]) : 0u;
            n_valid += __popc(__ballot_sync(FULL, valid));
            ok_min = min(ok_min, valid ? okey[e] : 0xFFFFu);
        }
        const float qc = nx_q;
        __syncwarp();
        if (lane < D) s_qb[wib][lane] = (unsigned short)(__float_as_uint(qc) >> 16);  // exact: the value came from bf16
        for (int t = lane; t < k; t += 32) row[t] = 0ull;
        fetch(r + stride);

        // the query's norms; error bound of the fp16 scores in the scaled units of the sweep
        float q2 = qc * qc, qa2 = lane < 16 ? qc * qc : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            q2 += __shfl_xor_sync(FULL, q2, o);
            qa2 += __shfl_xor_sync(FULL, qa2, o);
            ok_min = min(ok_min, __shfl_xor_sync(FULL, ok_min, o));
        }
        const F16HeadStat hs = stat[h];
        const float sq = f16_scale_from_n2max(hs.q_n2max), sk = f16_scale_from_n2max(hs.k_n2max);
        const float sc = sq * sk;  // scaled score = sc * score, a power of two
        const float nq = sqrtf(q2) * sq * 1.00001f, nqa = sqrtf(qa2) * sq * 1.00001f;
        const float nk = sqrtf(hs.k_n2max) * sk, nka = sqrtf(hs.k_first16_n2max) * sk;
        const float ea = f16_abs_err(KSTEPS, nqa, nka, nq, nk) * 1.0001f;
        const float er = kF16RelErr;
        const float fp32_err = 4e-6f * nq * nk;  // of the fp32 rescoring below, in scaled units
        const float g_min = __half2float(__ushort_as_half((unsigned short)f16_unordered(ok_min)));

        // m_k, the k-th largest group maximum: the largest 16-bit key that at least k entries reach, bit by bit
        float lowS = -CUDART_INF_F;
        if (n_valid >= k) {
            unsigned v = 0u;
#pragma unroll
            for (int bit = 15; bit >= 0; --bit) {
                const unsigned c = v | (1u << bit);
                int n = 0;
#pragma unroll
                for (int e = 0; e < EPL; ++e) n += __popc(__ballot_sync(FULL, okey[e] >= c));
                if (n >= k) v = c;
            }
            const float mk = __half2float(__ushort_as_half((unsigned short)f16_unordered(v)));
            lowS = mk - ea - er * fabsf(mk);
        }

        // groups that may hold one of the k best keys, compacted
        int n_kept = 0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const float g = __half2float(__ushort_as_half((unsigned short)f16_unordered(okey[e])));
            const bool keep = okey[e] != 0u && (g + ea + er * fabsf(g) >= lowS);
            const unsigned m = __ballot_sync(FULL, keep);
            if (keep) words[n_kept + __popc(m & ((1u << lane) - 1u))] = word[e];
            n_kept += __popc(m);
        }
        __syncwarp();

        // every key of the answer scores at least lowS / sc exactly; keep a margin for the fp32 sums
        const float floor_tau = n_valid >= k ? (lowS - fp32_err) / sc - 1e-30f : -CUDART_INF_F;
        float tau = floor_tau;
        int cnt = 0;
        // Rescoring, 32 keys (4 groups) per step.  A key row is P = D / 8 pieces of 16 bytes.  The rows come in by
        // asynchronous 16-byte copies in which P neighbouring lanes fetch one row, so one copy instruction touches
        // 32 / P cache lines instead of 32 (the kernel is bound by these line accesses); they land in a per-warp
        // stage of padded rows, one step ahead of the arithmetic.  Then each lane reads one whole row back and
        // scores it with the same chain of fused multiply-adds in index order as every other kernel.
        const int nsteps = (n_kept + 3) / 4;
        const unsigned char* kb = reinterpret_cast<const unsigned char*>(K) + ((size_t)h * D + pl * 8) * sizeof(T);
        auto issue = [&](int step) {
            if (step < nsteps) {
                unsigned char* buf = stage + (step & 1) * kStageBytes;
#pragma unroll
                for (int c = 0; c < P; ++c) {  // copy instruction c: keys c * 32 / P ... of the step
                    const int rrow = c * (32 / P) + lane / P;  // row of the stage = key of the step
                    const int t = step * 4 + (rrow >> 3);
                    if (t < n_kept) {
                        const uint32_t wd = words[t];
                        const int j = (int)(wd & 0x7FFFFFFFu) + (int)(wd >> 31) + 2 * (rrow & 7);
                        if (j < hi && kmip_check(j >= 0 && hi <= N, sb, 101))  // checks builds: key row inside K
                            ptx::cp_async_16(buf + rrow * kRowStride + pl * 16, kb + (size_t)(unsigned)j * row_bytes);
                    }
                }
            }
            ptx::cp_async_commit();  // an empty group when there is nothing left, so that the count below holds
        };
        uint32_t qp[D / 2];  // the query row, two bf16 values to a register
        __syncwarp();
#pragma unroll
        for (int v = 0; v < D / 8; ++v) {
            const uint4 t4 = *reinterpret_cast<const uint4*>(&s_qb[wib][v * 8]);
            qp[v * 4 + 0] = t4.x; qp[v * 4 + 1] = t4.y; qp[v * 4 + 2] = t4.z; qp[v * 4 + 3] = t4.w;
        }
        issue(0);
        for (int step = 0; step < nsteps; ++step) {
            issue(step + 1);
            ptx::cp_async_wait<1>();  // all but the newest group: this step's rows are in
            __syncwarp();
            const int t = step * 4 + (lane >> 3);
            const uint32_t wd = t < n_kept ? words[t] : 0u;
            const int jj = (int)(wd & 0x7FFFFFFFu) + (int)(wd >> 31) + 2 * (lane & 7);
            const bool kv = t < n_kept && jj < hi;
            float s = 0.0f;
            if (kv) {
                const unsigned char* kr = stage + (step & 1) * kStageBytes + lane * kRowStride;
#pragma unroll
                for (int v = 0; v < P; ++v) {
                    const uint4 rw = *reinterpret_cast<const uint4*>(kr + v * 16);
                    const uint32_t wv[4] = {rw.x, rw.y, rw.z, rw.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x) s = ptx::fma_bf16_pair(qp[v * 4 + x], wv[x], s);
                }
            }
            const bool pass = kv && (s > tau);
            const unsigned m = __ballot_sync(FULL, pass);
            if (m) {
                if (pass) row[k + cnt + __popc(m & ((1u << lane) - 1u))] = make_cand(s, jj);
                cnt += __popc(m);
                if (cnt > room - 32) {
                    // the groups come in list order, not key order: a later key with the same score as the
                    // k-th best and a smaller index must still get in, so the threshold sits just below it
                    tau = fmaxf(floor_tau, nextafterf(warp_merge_row_chunks(row, k, cnt, lane), -CUDART_INF_F));
                    cnt = 0;
                }
            }
            __syncwarp();  // the stage is free for the copies of step + 2
        }
        ptx::cp_async_wait<0>();
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
        __syncwarp();
    }
}

template <int D>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w) {
    const long long n_rows = (long long)a.N * a.H;
    const int blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
    constexpr int kSmem = kWarpsPerBlock * 2 * 32 * (D * 2 + 16);  // the rescoring stages
#define KMIP_LAUNCH_REFINE16(E_, LIST_) \
    if ((err = cudaFuncSetAttribute(refine_f16_kernel<D, E_, LIST_>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem)) != cudaSuccess) return err; \
    refine_f16_kernel<D, E_, LIST_><<<blocks, kWarpsPerBlock * 32, kSmem, a.stream>>>( \
        static_cast<const __nv_bfloat16*>(a.Q), static_cast<const __nv_bfloat16*>(a.K), a.graph_offsets, a.G, (int)a.N, \
        a.H, a.k, reinterpret_cast<const uint32_t*>(a.ws + w.cand_word_off), \
        reinterpret_cast<const uint16_t*>(a.ws + w.cand_half_off), reinterpret_cast<const F16HeadStat*>(a.ws + w.f16stat_off), \
        a.topk_idx, a.topk_score, reinterpret_cast<StatusBlock*>(a.ws), reinterpret_cast<int*>(a.ws + w.redo_off))
    cudaError_t err;
    // the list sizes are those of score_select_f16_list
    if (a.k <= 8) { KMIP_LAUNCH_REFINE16(2, 16); }
    else if (a.k <= 16) { KMIP_LAUNCH_REFINE16(2, 24); }
    else { KMIP_LAUNCH_REFINE16(4, kF16List32); }
#undef KMIP_LAUNCH_REFINE16
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_refine_f16(const FwdArgs& a, const FwdWorkspace& w) {
    return a.d == 16 ? launch_d<16>(a, w) : launch_d<32>(a, w);
}

}  // namespace kmip
