// Sparse backward of k-MIP attention with the selection held constant (Sec. 3.1: the top-k
// indices are reused; App. E: I_argtopk and E_topk need no recomputation).
//
//   rows      per (query, head): p = softmax(E_topk / sqrt(d)), dP_t = g . v_t, D = sum p dP,
//             dS_t = p_t (dP_t - D) / sqrt(d), dQ = sum_t dS_t k_t; p and dS go to scratch.
//   inverse   key-major index of the selected pairs: histogram of hits per (key, head),
//             exclusive scan, scatter of pair ids.
//   segments  per (key, head): dV = sum p g_i, dK = sum dS q_i over its hit list; lists longer
//             than kLongSeg (hub keys) are reduced by a whole block each.
#include <algorithm>

#include "common.cuh"
#include "rowops.cuh"

namespace kmip {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kLongSeg = 512;

// ------------------------------------------------------------------------------------------ rows
template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_rows_kernel(const T* __restrict__ K, const T* __restrict__ V, const T* __restrict__ dOut,
                const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_score,
                int N, int H, int k, float scale, float drop_p, unsigned long long seed,
                float* __restrict__ ws_p, float* __restrict__ ws_ds, T* __restrict__ dQ) {
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

        // dP_t = g_i . v_{j_t}: each lane owns its entries and walks the d columns
        float dP[kMaxEntriesPerLane];
#pragma unroll
        for (int e = 0; e < kMaxEntriesPerLane; ++e) dP[e] = 0.0f;
        const T* g = dOut + (size_t)r * D;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += VEC) {
            float gv[VEC];
            Elem<T>::load_vec(g + c0, gv);
#pragma unroll
            for (int e = 0; e < kMaxEntriesPerLane; ++e) {
                if (e * 32 < k && j[e] >= 0) {
                    float vv[VEC];
                    Elem<T>::load_vec(V + ((size_t)j[e] * H + h) * D + c0, vv);
#pragma unroll
                    for (int c = 0; c < VEC; ++c) dP[e] = fmaf(gv[c], vv[c], dP[e]);
                }
            }
        }
        // with dropout the output was sum_t f_t p_t v_t (f constant here): dP_t = f_t (g . v_t), and the
        // weight that reaches dV is f_t p_t
        float f[kMaxEntriesPerLane];
#pragma unroll
        for (int e = 0; e < kMaxEntriesPerLane; ++e) f[e] = 1.0f;
        if (drop_p > 0.0f) {
            dropout_factors(r, k, lane, drop_p, seed, f);
#pragma unroll
            for (int e = 0; e < kMaxEntriesPerLane; ++e) dP[e] *= f[e];
        }
        float dsum = 0.0f;
#pragma unroll
        for (int e = 0; e < kMaxEntriesPerLane; ++e) dsum = fmaf(p[e], dP[e], dsum);
        dsum = warp_sum(dsum);
        float dS[kMaxEntriesPerLane];
#pragma unroll
        for (int e = 0; e < kMaxEntriesPerLane; ++e) {
            dS[e] = scale * p[e] * (dP[e] - dsum);
            const int t = e * 32 + lane;
            if (t < k) {
                ws_p[(size_t)r * k + t] = f[e] * p[e];
                ws_ds[(size_t)r * k + t] = dS[e];
            }
        }
        float acc[VEC];
        gather_weighted_sum<T, D>(K, H, h, k, lane, j, dS, acc);
        if (lane < LPR) Elem<T>::store_vec(dQ + (size_t)r * D + lane * VEC, acc);
    }
}

// --------------------------------------------------------------------------------------- inverse
__global__ void hist_kernel(const int32_t* __restrict__ topk_idx, long long n_pairs, int N, int H, int k,
                            int* __restrict__ counts, StatusBlock* __restrict__ sb) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_pairs) return;
    const int j = __ldg(topk_idx + e);
    kmip_check(j < N, sb, 105);  // checks builds: an index the forward pass cannot have written (ignored either way)
    if (j < 0 || j >= N) return;
    const int h = (int)((e / k) % H);
    atomicAdd(counts + (size_t)j * H + h, 1);
}

__device__ inline int block_reduce_sum_1024(int v, int* s_warp) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    if (lane == 0) s_warp[wid] = v;
    __syncthreads();
    int t = (threadIdx.x < 32) ? s_warp[threadIdx.x] : 0;
    if (wid == 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
        if (lane == 0) s_warp[0] = t;
    }
    __syncthreads();
    const int r = s_warp[0];
    __syncthreads();
    return r;
}

// exclusive scan of one value per thread over a 1024-thread block; returns the block total in `total`
__device__ inline int block_exclusive_scan_1024(int v, int* s_warp, int& total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        int w = s_warp[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, w, o);
            if (lane >= o) w += t;
        }
        s_warp[lane] = w;
    }
    __syncthreads();
    const int base = wid ? s_warp[wid - 1] : 0;
    total = s_warp[31];
    __syncthreads();
    return base + incl - v;
}

constexpr int kScanThreads = 1024;
constexpr int kScanPerThread = kScanItemsPerBlock / kScanThreads;  // 4

__global__ void __launch_bounds__(kScanThreads)
scan_block_sums_kernel(const int* __restrict__ counts, long long n, int* __restrict__ block_sums) {
    __shared__ int s_warp[32];
    const long long base = (long long)blockIdx.x * kScanItemsPerBlock + (long long)threadIdx.x * kScanPerThread;
    int v = 0;
#pragma unroll
    for (int u = 0; u < kScanPerThread; ++u)
        if (base + u < n) v += counts[base + u];
    const int s = block_reduce_sum_1024(v, s_warp);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = s;
}

__global__ void __launch_bounds__(kScanThreads)
scan_block_offsets_kernel(int* __restrict__ block_sums, int n_blocks) {
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int b0 = 0; b0 < n_blocks; b0 += kScanThreads) {
        const int b = b0 + threadIdx.x;
        const int v = b < n_blocks ? block_sums[b] : 0;
        int total;
        const int ex = block_exclusive_scan_1024(v, s_warp, total);
        if (b < n_blocks) block_sums[b] = s_carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) s_carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) block_sums[n_blocks] = s_carry;
}

// Writes the exclusive offsets, resets the counters (they become fill cursors) and lists the
// segments that are long enough to deserve a whole block.
__global__ void __launch_bounds__(kScanThreads)
scan_write_kernel(int* __restrict__ counts, long long n, const int* __restrict__ block_sums,
                  int* __restrict__ seg_off, int* __restrict__ long_list, StatusBlock* __restrict__ sb) {
    __shared__ int s_warp[32];
    const long long base = (long long)blockIdx.x * kScanItemsPerBlock + (long long)threadIdx.x * kScanPerThread;
    int c[kScanPerThread];
    int v = 0;
#pragma unroll
    for (int u = 0; u < kScanPerThread; ++u) {
        c[u] = (base + u < n) ? counts[base + u] : 0;
        v += c[u];
    }
    int total;
    int off = block_sums[blockIdx.x] + block_exclusive_scan_1024(v, s_warp, total);
#pragma unroll
    for (int u = 0; u < kScanPerThread; ++u) {
        if (base + u < n) {
            seg_off[base + u] = off;
            counts[base + u] = 0;
            if (c[u] > kLongSeg) long_list[atomicAdd(&sb->n_long, 1)] = (int)(base + u);
        } else if (base + u == n) {
            seg_off[n] = off;
        }
        off += c[u];
    }
}

// A hit record of the key-major lists: everything the segment reduction needs about one selected
// pair in one 16-byte load - the query row, its softmax weight p (times the dropout factor) and its
// score gradient dS - instead of a pair id that would cost two more scattered 4-byte reads per hit.
__global__ void fill_kernel(const int32_t* __restrict__ topk_idx, long long n_pairs, int N, int H, int k,
                            const float* __restrict__ ws_p, const float* __restrict__ ws_ds,
                            const int* __restrict__ seg_off, int* __restrict__ cursor, int4* __restrict__ hits,
                            StatusBlock* __restrict__ sb) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_pairs) return;
    const int j = __ldg(topk_idx + e);
    if (j < 0 || j >= N) return;
    const long long r = e / k;  // query * H + head
    const int h = (int)(r % H);
    const size_t key = (size_t)j * H + h;
    const long long pos = (long long)seg_off[key] + atomicAdd(cursor + key, 1);
    if (!kmip_check(pos >= 0 && pos < n_pairs, sb, 104)) return;  // checks builds: inside the hit lists
    hits[pos] =
        make_int4((int)(r / H), __float_as_int(__ldg(ws_p + e)), __float_as_int(__ldg(ws_ds + e)), 0);
}

// -------------------------------------------------------------------------------------- segments
// Accumulate one hit into the lane's part of dV and dK.
template <typename T, int D>
__device__ __forceinline__ void accumulate_hit(int4 rec, int h, int H, int part,
                                               const T* __restrict__ Q, const T* __restrict__ dOut,
                                               float (&accV)[Elem<T>::kVec], float (&accK)[Elem<T>::kVec]) {
    constexpr int VEC = Elem<T>::kVec;
    const float pw = __int_as_float(rec.y), dsw = __int_as_float(rec.z);
    const size_t off = ((size_t)rec.x * H + h) * D + part * VEC;
    float gv[VEC], qv[VEC];
    Elem<T>::load_vec(dOut + off, gv);
    Elem<T>::load_vec(Q + off, qv);
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        accV[c] = fmaf(pw, gv[c], accV[c]);
        accK[c] = fmaf(dsw, qv[c], accK[c]);
    }
}

// Accumulates the hits first, first+stride, ... (< len) of one list; four hits are in flight at a time
// so that the dependent loads (record -> rows) of different hits overlap.
template <typename T, int D>
__device__ __forceinline__ void accumulate_list(const int4* __restrict__ list, int first, int stride, int len,
                                                int h, int H, int part, const T* __restrict__ Q,
                                                const T* __restrict__ dOut, float (&accV)[Elem<T>::kVec],
                                                float (&accK)[Elem<T>::kVec]) {
    constexpr int VEC = Elem<T>::kVec;
    int t = first;
    for (; t + 3 * stride < len; t += 4 * stride) {
        int4 rec[4];
        float gv[4][VEC], qv[4][VEC];
#pragma unroll
        for (int u = 0; u < 4; ++u) rec[u] = __ldg(list + t + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t off = ((size_t)rec[u].x * H + h) * D + part * VEC;
            Elem<T>::load_vec(dOut + off, gv[u]);
            Elem<T>::load_vec(Q + off, qv[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float pw = __int_as_float(rec[u].y), dsw = __int_as_float(rec[u].z);
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                accV[c] = fmaf(pw, gv[u][c], accV[c]);
                accK[c] = fmaf(dsw, qv[u][c], accK[c]);
            }
        }
    }
    for (; t < len; t += stride) accumulate_hit<T, D>(__ldg(list + t), h, H, part, Q, dOut, accV, accK);
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_segments_kernel(const T* __restrict__ Q, const T* __restrict__ dOut,
                    const int* __restrict__ seg_off, const int4* __restrict__ hits,
                    long long n_segs, int H, int k, T* __restrict__ dK, T* __restrict__ dV) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int EPW = 32 / LPR;
    const int lane = threadIdx.x & 31, part = lane % LPR, sub = lane / LPR;
    for (long long x = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); x < n_segs;
         x += (long long)gridDim.x * kWarpsPerBlock) {
        const int start = __ldg(seg_off + x), len = __ldg(seg_off + x + 1) - start;
        if (len > kLongSeg) continue;  // reduced by bwd_long_segments_kernel
        const int h = (int)(x % H);
        float accV[VEC], accK[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) { accV[c] = 0.0f; accK[c] = 0.0f; }
        accumulate_list<T, D>(hits + start, sub, EPW, len, h, H, part, Q, dOut, accV, accK);
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                accV[c] += __shfl_xor_sync(0xFFFFFFFFu, accV[c], o);
                accK[c] += __shfl_xor_sync(0xFFFFFFFFu, accK[c], o);
            }
        }
        if (lane < LPR) {
            Elem<T>::store_vec(dV + (size_t)x * D + lane * VEC, accV);
            Elem<T>::store_vec(dK + (size_t)x * D + lane * VEC, accK);
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_long_segments_kernel(const T* __restrict__ Q, const T* __restrict__ dOut,
                         const int* __restrict__ seg_off, const int4* __restrict__ hits,
                         const int* __restrict__ long_list, const StatusBlock* __restrict__ sb,
                         int H, int k, T* __restrict__ dK, T* __restrict__ dV) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int EPW = 32 / LPR;
    __shared__ float s_part[kWarpsPerBlock][2][D];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, part = lane % LPR, sub = lane / LPR;
    const int n_long = sb->n_long;
    // Head by head: the dO and Q rows of one head (N * d elements each) fit the L2 cache, those of
    // all heads together do not, and a query row is gathered k times across the lists of a head.
    for (int hp = 0; hp < H; ++hp)
    for (int li = blockIdx.x; li < n_long; li += gridDim.x) {
        const int x = __ldg(long_list + li);
        const int h = x % H;
        if (h != hp) continue;  // block-uniform
        const int start = __ldg(seg_off + x), len = __ldg(seg_off + x + 1) - start;
        float accV[VEC], accK[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) { accV[c] = 0.0f; accK[c] = 0.0f; }
        accumulate_list<T, D>(hits + start, wid * EPW + sub, kWarpsPerBlock * EPW, len, h, H, part, Q, dOut, accV, accK);
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                accV[c] += __shfl_xor_sync(0xFFFFFFFFu, accV[c], o);
                accK[c] += __shfl_xor_sync(0xFFFFFFFFu, accK[c], o);
            }
        }
        __syncthreads();  // previous segment's readers are done with s_part
        if (lane < LPR) {
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                s_part[wid][0][lane * VEC + c] = accV[c];
                s_part[wid][1][lane * VEC + c] = accK[c];
            }
        }
        __syncthreads();
        if (wid == 0 && lane < LPR) {
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                float sv = 0.0f, sk = 0.0f;
#pragma unroll
                for (int w = 0; w < kWarpsPerBlock; ++w) {
                    sv += s_part[w][0][lane * VEC + c];
                    sk += s_part[w][1][lane * VEC + c];
                }
                accV[c] = sv;
                accK[c] = sk;
            }
            Elem<T>::store_vec(dV + (size_t)x * D + lane * VEC, accV);
            Elem<T>::store_vec(dK + (size_t)x * D + lane * VEC, accK);
        }
    }
}

// -------------------------------------------------------------------------------------- launcher
template <typename T, int D>
cudaError_t launch_d(const BwdArgs& a, const BwdWorkspace& w, cudaEvent_t* ev) {
    const long long n_rows = (long long)a.N * a.H, n_pairs = n_rows * a.k;
    StatusBlock* sb = reinterpret_cast<StatusBlock*>(a.ws);
    float* ws_p = reinterpret_cast<float*>(a.ws + w.p_off);
    float* ws_ds = reinterpret_cast<float*>(a.ws + w.ds_off);
    int* seg_off = reinterpret_cast<int*>(a.ws + w.seg_off);
    int* cursor = reinterpret_cast<int*>(a.ws + w.cursor_off);
    int4* hits = reinterpret_cast<int4*>(a.ws + w.pairs_off);
    int* block_sums = reinterpret_cast<int*>(a.ws + w.blocksum_off);
    int* long_list = reinterpret_cast<int*>(a.ws + w.long_off);
    const T *Q = static_cast<const T*>(a.Q), *K = static_cast<const T*>(a.K), *V = static_cast<const T*>(a.V);
    const T* dOut = static_cast<const T*>(a.d_out);
    const float scale = 1.0f / sqrtf((float)a.d);
    cudaError_t err;

    if ((err = cudaMemsetAsync(cursor, 0, sizeof(int) * (size_t)(n_rows + 1), a.stream)) != cudaSuccess) return err;

    const int row_blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
    bwd_rows_kernel<T, D><<<row_blocks, kWarpsPerBlock * 32, 0, a.stream>>>(
        K, V, dOut, a.topk_idx, a.topk_score, (int)a.N, a.H, a.k, scale, a.drop_p, a.seed, ws_p, ws_ds,
        static_cast<T*>(a.dQ));
    if (ev) cudaEventRecord(ev[0], a.stream);

    const int pair_blocks = (int)((n_pairs + 255) / 256);
    hist_kernel<<<pair_blocks, 256, 0, a.stream>>>(a.topk_idx, n_pairs, (int)a.N, a.H, a.k, cursor, sb);
    scan_block_sums_kernel<<<w.scan_blocks, kScanThreads, 0, a.stream>>>(cursor, n_rows, block_sums);
    scan_block_offsets_kernel<<<1, kScanThreads, 0, a.stream>>>(block_sums, w.scan_blocks);
    scan_write_kernel<<<w.scan_blocks, kScanThreads, 0, a.stream>>>(cursor, n_rows, block_sums, seg_off, long_list, sb);
    fill_kernel<<<pair_blocks, 256, 0, a.stream>>>(a.topk_idx, n_pairs, (int)a.N, a.H, a.k, ws_p, ws_ds, seg_off, cursor,
                                                  hits, sb);
    if (ev) cudaEventRecord(ev[1], a.stream);

    bwd_segments_kernel<T, D><<<row_blocks, kWarpsPerBlock * 32, 0, a.stream>>>(
        Q, dOut, seg_off, hits, n_rows, a.H, a.k, static_cast<T*>(a.dK), static_cast<T*>(a.dV));
    bwd_long_segments_kernel<T, D><<<sm_count() * 8, kWarpsPerBlock * 32, 0, a.stream>>>(
        Q, dOut, seg_off, hits, long_list, sb, a.H, a.k, static_cast<T*>(a.dK), static_cast<T*>(a.dV));
    if (ev) cudaEventRecord(ev[2], a.stream);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(const BwdArgs& a, const BwdWorkspace& w, cudaEvent_t* ev) {
    switch (a.d) {
        case 16: return launch_d<T, 16>(a, w, ev);
        case 32: return launch_d<T, 32>(a, w, ev);
        case 64: return launch_d<T, 64>(a, w, ev);
        case 128: return launch_d<T, 128>(a, w, ev);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_backward(const BwdArgs& a, const BwdWorkspace& w, cudaEvent_t* ev) {
    return a.mode == KMIP_FP32_EXACT ? launch_t<float>(a, w, ev) : launch_t<__nv_bfloat16>(a, w, ev);
}

}  // namespace kmip
