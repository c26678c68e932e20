// Query reordering for the tensor-core sweep (not in the paper; exact by the permutation
// equivariance of self-attention, Sec. 3).
//
// In the sweep a warp owns 32 query rows, and a key tile costs the whole warp its candidate path
// as soon as ONE of those rows has a group above its threshold.  Rows with similar queries have
// their hits in the same key tiles, so the sweep runs the rows of a graph in an order that puts
// similar queries next to each other: every node gets a 12-bit sign code of its query vector
// (all heads) against 12 fixed pseudo-random +-1 directions, and the rows of each large graph are
// bucket-sorted by that code.  The sweep reads a row-permuted copy of Q and writes each row's
// result back to the row's own place; nothing else sees the permutation.  On point-cloud-like data
// (queries in tight clusters) this removes about a tenth of the sweep time; on unstructured data
// it changes nothing.
//
// The pruned sweep (prune.cu) also orders the KEYS of large graphs, by (norm class, nearest pivot), and
// takes the query codes from the same pivots; see pivot_code_kernel below.
#include <algorithm>

#include "common.cuh"

namespace kmip {

namespace {

constexpr int kCodeBits = 12;       // query codes
constexpr int kSortThreads = 1024;

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
    return x;
}

// One warp per node: bit b of the code is the sign of sum_c s(b, c) * q_c over the H*d columns of
// the node's query row, s(b, c) = +-1 from bit b of a hash of c.
__global__ void query_code_kernel(const __nv_bfloat16* __restrict__ Q, int N, int HD, unsigned short* __restrict__ code,
                                  const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= N) return;
    float acc[kCodeBits];
#pragma unroll
    for (int b = 0; b < kCodeBits; ++b) acc[b] = 0.0f;
    for (int c = lane; c < HD; c += 32) {
        const float x = Elem<__nv_bfloat16>::load(Q + (size_t)row * HD + c);
        const uint32_t m = mix32((uint32_t)c + 0x9E3779B9u);
#pragma unroll
        for (int b = 0; b < kCodeBits; ++b) acc[b] += ((m >> b) & 1u) ? x : -x;
    }
    unsigned bits = 0;
#pragma unroll
    for (int b = 0; b < kCodeBits; ++b) {
        float v = acc[b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        bits |= (v > 0.0f ? 1u : 0u) << b;
    }
    if (lane == 0) code[row] = (unsigned short)bits;
}

// One block per graph: counting sort of the graph's rows by code (any order inside a bucket).
// perm[sorted position] = original row; both lie in the graph's own row range.
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
graph_sort_kernel(const int32_t* __restrict__ offs, int G, int N, const unsigned short* __restrict__ code,
                  int* __restrict__ perm, const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;  // malformed offsets were reported by the plan kernel
    constexpr int kBuckets = 1 << BITS;
    constexpr int PER = kBuckets >= kSortThreads ? kBuckets / kSortThreads : 1;  // consecutive bins per thread in the scan
    extern __shared__ int s_bin[];
    __shared__ int s_warp[32];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int n_graphs = offs ? G : 1;
    for (int g = blockIdx.x; g < n_graphs; g += gridDim.x) {
        const int lo = offs ? __ldg(offs + g) : 0, hi = offs ? __ldg(offs + g + 1) : N;
        if (hi - lo < kMinRowsToSort) {
            for (int r = lo + tid; r < hi; r += kSortThreads) perm[r] = r;
            continue;
        }
        __syncthreads();  // the previous graph's cursors are no longer needed
        for (int b = tid; b < kBuckets; b += kSortThreads) s_bin[b] = 0;
        __syncthreads();
        for (int r = lo + tid; r < hi; r += kSortThreads) atomicAdd(&s_bin[code[r]], 1);
        __syncthreads();
        // exclusive scan of the counts: PER consecutive bins per thread
        int c[PER], sum = 0;
#pragma unroll
        for (int x = 0; x < PER; ++x) { c[x] = tid * PER + x < kBuckets ? s_bin[tid * PER + x] : 0; sum += c[x]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            int v = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, v, o);
                if (lane >= o) v += t;
            }
            s_warp[lane] = v;  // inclusive over warps
        }
        __syncthreads();
        int start = lo + (wid ? s_warp[wid - 1] : 0) + incl - sum;
#pragma unroll
        for (int x = 0; x < PER; ++x)
            if (tid * PER + x < kBuckets) { s_bin[tid * PER + x] = start; start += c[x]; }
        __syncthreads();
        for (int r = lo + tid; r < hi; r += kSortThreads) perm[atomicAdd(&s_bin[code[r]], 1)] = r;
    }
}

// The same sort, but stable (rows of a bucket stay in row order), so that the order - and with it which of
// several keys with exactly equal scores the pruned sweep meets first - does not depend on the timing of
// atomics.  Each of the 32 warps owns a contiguous chunk of the graph's rows and a histogram row of its
// own in shared memory; after the counts are turned into start positions per (warp, bucket), a warp places
// its rows 32 at a time, ranking equal codes inside the 32 with a match vote.  32 * 2^BITS counters:
// BITS <= 10.
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
graph_sort_stable_kernel(const int32_t* __restrict__ offs, int G, int N, const unsigned short* __restrict__ code,
                         int* __restrict__ perm, const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    constexpr int kBuckets = 1 << BITS;
    constexpr int kWarpsS = kSortThreads / 32;
    static_assert(kBuckets <= kSortThreads, "one thread per bucket in the scan");
    extern __shared__ int s_hist[];  // [kWarpsS][kBuckets]
    __shared__ int s_warp[32];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int n_graphs = offs ? G : 1;
    for (int g = blockIdx.x; g < n_graphs; g += gridDim.x) {
        const int lo = offs ? __ldg(offs + g) : 0, hi = offs ? __ldg(offs + g + 1) : N;
        if (hi - lo < kMinRowsToSort) {
            for (int r = lo + tid; r < hi; r += kSortThreads) perm[r] = r;
            continue;
        }
        __syncthreads();
        for (int x = tid; x < kWarpsS * kBuckets; x += kSortThreads) s_hist[x] = 0;
        __syncthreads();
        const int chunk = (hi - lo + kWarpsS - 1) / kWarpsS;
        const int c_lo = min(hi, lo + wid * chunk), c_hi = min(hi, c_lo + chunk);
        int* mine = s_hist + wid * kBuckets;
        for (int r = c_lo + lane; r < c_hi; r += 32) atomicAdd(&mine[code[r]], 1);  // contention inside the warp only
        __syncthreads();
        // thread b < kBuckets: total of bucket b, exclusive scan over buckets, then start of every warp's share
        int total = 0;
        if (tid < kBuckets)
            for (int w = 0; w < kWarpsS; ++w) total += s_hist[w * kBuckets + tid];
        int incl = total;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            int v = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, v, o);
                if (lane >= o) v += t;
            }
            s_warp[lane] = v;
        }
        __syncthreads();
        if (tid < kBuckets) {
            int start = lo + (wid ? s_warp[wid - 1] : 0) + incl - total;
            for (int w = 0; w < kWarpsS; ++w) {
                const int c = s_hist[w * kBuckets + tid];
                s_hist[w * kBuckets + tid] = start;
                start += c;
            }
        }
        __syncthreads();
        for (int r0 = c_lo; r0 < c_hi; r0 += 32) {
            const int r = r0 + lane;
            const bool live = r < c_hi;
            const unsigned cd = live ? code[r] : 0xFFFFFFFFu;  // idle lanes match among themselves only
            const unsigned same = __match_any_sync(0xFFFFFFFFu, cd);
            if (live) {
                const int rank = __popc(same & ((1u << lane) - 1u));
                perm[mine[cd] + rank] = r;
            }
            __syncwarp();
            if (live && (same >> lane) == 1u) mine[cd] += __popc(same);  // the group's highest lane moves the cursor
            __syncwarp();
        }
    }
}

// Qp[p, :] = Q[perm[p], :], 16 bytes per thread.
__global__ void gather_rows_kernel(const uint4* __restrict__ Q, const int* __restrict__ perm, uint4* __restrict__ Qp,
                                   long long n_vec, int vec_per_row, const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const long long p = v / vec_per_row;
    const int c = (int)(v % vec_per_row);
    Qp[v] = __ldg(Q + (long long)__ldg(perm + p) * vec_per_row + c);
}


// ---- keys of the pruned sweep -------------------------------------------------------------------
__device__ inline int graph_of(const int32_t* offs, int G, int i) {
    if (offs == nullptr) return 0;
    int a = 0, b = G;
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (__ldg(offs + m) <= i) a = m; else b = m;
    }
    return a;
}

// One warp per node: squared norm of the whole key vector, and the largest of each graph.
__global__ void key_norm_kernel(const __nv_bfloat16* __restrict__ K, int N, int HD, const int32_t* __restrict__ offs,
                                int G, float* __restrict__ norm2, unsigned* __restrict__ gmax,
                                const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= N) return;
    float s = 0.0f;
    for (int c = lane; c < HD; c += 32) {
        const float x = Elem<__nv_bfloat16>::load(K + (size_t)row * HD + c);
        s = fmaf(x, x, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (!(s >= 0.0f && s <= 3.0e38f)) s = 3.0e38f;  // NaN or overflow: treated as the largest class
    if (lane == 0) {
        norm2[row] = s;
        atomicMax(gmax + graph_of(offs, G, (int)row), __float_as_uint(s));  // non-negative floats order like their bits
    }
}

// Pivot codes.  Every large graph takes kPivots of its key rows (evenly spaced) as pivots; a key's code is
// its nearest pivot (largest k.p - |p|^2/2), a query's code the pivot with the largest inner product q.p,
// i.e. the part of the key set its best keys are expected in.  Rows that share a pivot are similar, so
// sorting by the code makes the 128-row tiles tight, which is what the centroid bound needs; and a block
// of queries can start its sweep at its own pivot's keys.  A key's code carries its norm class in front:
// 0 within a factor 2 of the graph's largest key norm, 1 within 4, 2 within 8, 3 the rest.
// One block per work item (rows of one graph); 8 warps, four rows per warp and step, the pivots in
// shared memory as fp32 with an odd row pitch (lane p reads pivot p: no bank conflicts).  Vectors wider
// than 64 are compared on 64 evenly spaced columns.
constexpr int kPivots = 256;
constexpr int kPivotDims = 64;  // columns compared (evenly spaced when the vector is wider)
constexpr int kPivotBits = 8;
constexpr int kKeyCodeBits2 = kPivotBits + 2;
constexpr int kAssignThreads = 256;

template <bool KEYS>
__global__ void __launch_bounds__(kAssignThreads)
pivot_code_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ K, int HD,
                  const WorkItem* __restrict__ items, const StatusBlock* __restrict__ sb,
                  const int32_t* __restrict__ offs, int G, const float* __restrict__ norm2,
                  const unsigned* __restrict__ gmax, unsigned short* __restrict__ code) {
    if (sb->status != KMIP_OK) return;
    if ((int)blockIdx.x >= sb->n_items) return;
    const WorkItem it = items[blockIdx.x];
    const int n = it.key_hi - it.key_lo;
    if (n < kMinRowsToSort) return;  // the graph keeps its order; its codes are never read
    const int DP = min(HD, kPivotDims), pitch = DP + 1;
    extern __shared__ float s_piv[];           // [kPivots][pitch]
    float* s_bias = s_piv + kPivots * pitch;   // [kPivots]
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    for (int x = tid; x < kPivots * DP; x += kAssignThreads) {
        const int p = x / DP, c = x % DP;
        const long long row = it.key_lo + (long long)p * n / kPivots;
        s_piv[p * pitch + c] = Elem<__nv_bfloat16>::load(K + (size_t)row * HD + (size_t)c * HD / DP);
    }
    __syncthreads();
    for (int p = tid; p < kPivots; p += kAssignThreads) {
        float t = 0.0f;
        for (int c = 0; c < DP; ++c) t = fmaf(s_piv[p * pitch + c], s_piv[p * pitch + c], t);
        s_bias[p] = KEYS ? -0.5f * t : 0.0f;
    }
    __syncthreads();
    float mx = 0.0f;
    if (KEYS) mx = __uint_as_float(__ldg(gmax + graph_of(offs, G, it.key_lo)));
    constexpr int R = 4;  // rows per warp and step: every pivot value read from shared memory serves R rows
    for (int r0 = wid * R; r0 < it.nrows; r0 += (kAssignThreads / 32) * R) {
        float x[R][2];
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const int row = it.row0 + min(r0 + q, it.nrows - 1);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int c = lane + 32 * i;
                x[q][i] = c < DP ? Elem<__nv_bfloat16>::load(X + (size_t)row * HD + (size_t)c * HD / DP) : 0.0f;
            }
        }
        float sc[R][kPivots / 32];
#pragma unroll
        for (int j = 0; j < kPivots / 32; ++j) {
            const float bias = s_bias[lane + 32 * j];
#pragma unroll
            for (int q = 0; q < R; ++q) sc[q][j] = bias;
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            if (32 * i >= DP) break;
            const int cn = min(32, DP - 32 * i);
            for (int cc = 0; cc < cn; ++cc) {
                float v[R];
#pragma unroll
                for (int q = 0; q < R; ++q) v[q] = __shfl_sync(0xFFFFFFFFu, x[q][i], cc);
                const float* col = s_piv + lane * pitch + 32 * i + cc;
#pragma unroll
                for (int j = 0; j < kPivots / 32; ++j) {
                    const float pv = col[32 * j * pitch];
#pragma unroll
                    for (int q = 0; q < R; ++q) sc[q][j] = fmaf(v[q], pv, sc[q][j]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < R; ++q) {
            float best = sc[q][0];
            int bi = lane;
#pragma unroll
            for (int j = 1; j < kPivots / 32; ++j)
                if (sc[q][j] > best) { best = sc[q][j]; bi = lane + 32 * j; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
                const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
                if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
            if (lane == 0 && r0 + q < it.nrows) {
                const int row = it.row0 + r0 + q;
                unsigned cls = 0;
                if (KEYS) {
                    const float n2 = norm2[row];
                    cls = n2 * 4.0f >= mx ? 0u : n2 * 16.0f >= mx ? 1u : n2 * 64.0f >= mx ? 2u : 3u;
                }
                code[row] = (unsigned short)((cls << kPivotBits) | (unsigned)bi);
            }
        }
    }
}

// Kp[h, p, :] = K[kperm[p], h, :], 16 bytes per thread.
__global__ void pack_keys_perm_kernel(const uint4* __restrict__ K, const int* __restrict__ kperm, uint4* __restrict__ Kp,
                                      long long n_vec, int N, int H, int vec_per_row, const StatusBlock* __restrict__ sb,
                                      const unsigned short* __restrict__ code, unsigned short* __restrict__ code_sorted) {
    if (sb->status != KMIP_OK) return;
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const long long ph = v / vec_per_row;  // p * H + h
    const int c = (int)(v % vec_per_row);
    const long long p = ph / H;
    const int h = (int)(ph % H);
    const int src = __ldg(kperm + p);
    Kp[((long long)h * N + p) * vec_per_row + c] = __ldg(K + ((long long)src * H + h) * vec_per_row + c);
    if (h == 0 && c == 0) code_sorted[p] = code[src];  // the codes in sweep order (start tile of a query block)
}

}  // namespace

// After launch_plan (which validates the offsets): codes, per-graph bucket sort, permuted copy of Q.
cudaError_t launch_reorder_queries(const FwdArgs& a, const FwdWorkspace& w) {
    const StatusBlock* sb = reinterpret_cast<const StatusBlock*>(a.ws);
    unsigned short* code = reinterpret_cast<unsigned short*>(a.ws + w.code_off);
    int* perm = reinterpret_cast<int*>(a.ws + w.perm_off);
    const int HD = a.H * a.d;
    const int n_graphs = a.graph_offsets ? a.G : 1;
    if (w.prune) {
        // pruned sweep: a query's code is the key pivot it scores highest against
        const int DP = std::min(HD, kPivotDims);
        const int smem = (kPivots * (DP + 1) + kPivots) * 4;
        auto kern = pivot_code_kernel<false>;
        cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (err != cudaSuccess) return err;
        kern<<<w.max_items, kAssignThreads, smem, a.stream>>>(
            static_cast<const __nv_bfloat16*>(a.Q), static_cast<const __nv_bfloat16*>(a.K), HD,
            reinterpret_cast<const WorkItem*>(a.ws + w.items_off), sb, a.graph_offsets, a.G, nullptr, nullptr, code);
        graph_sort_stable_kernel<kPivotBits><<<std::min(n_graphs, sm_count() * 2), kSortThreads, (32 << kPivotBits) * 4, a.stream>>>(
            a.graph_offsets, a.G, (int)a.N, code, perm, sb);
    } else {
        query_code_kernel<<<(unsigned)((a.N * 32 + 255) / 256), 256, 0, a.stream>>>(
            static_cast<const __nv_bfloat16*>(a.Q), (int)a.N, HD, code, sb);
        graph_sort_kernel<kCodeBits><<<std::min(n_graphs, sm_count() * 2), kSortThreads, (1 << kCodeBits) * 4, a.stream>>>(
            a.graph_offsets, a.G, (int)a.N, code, perm, sb);
    }
    if (w.f16) return cudaGetLastError();  // the half-precision prefilter gathers while it converts (f16_convert.cu)
    const int vec_per_row = HD * 2 / 16;
    const long long n_vec = (long long)a.N * vec_per_row;
    gather_rows_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.Q), perm, reinterpret_cast<uint4*>(a.ws + w.qperm_off), n_vec, vec_per_row, sb);
    return cudaGetLastError();
}

// Pruned sweep: per-graph sort of the keys by (norm class, locality code) and the regrouped copy of K in
// that order.  Uses the code buffer after launch_reorder_queries is done with it (same stream).
cudaError_t launch_reorder_keys(const FwdArgs& a, const FwdWorkspace& w) {
    const StatusBlock* sb = reinterpret_cast<const StatusBlock*>(a.ws);
    unsigned short* code = reinterpret_cast<unsigned short*>(a.ws + w.kcode_off);
    unsigned short* code_sorted = reinterpret_cast<unsigned short*>(a.ws + w.kcs_off);
    int* kperm = reinterpret_cast<int*>(a.ws + w.kperm_off);
    float* norm2 = reinterpret_cast<float*>(a.ws + w.knorm_off);
    unsigned* gmax = reinterpret_cast<unsigned*>(a.ws + w.gmax_off);
    const int HD = a.H * a.d;
    const int n_graphs = a.graph_offsets ? a.G : 1;
    cudaError_t err = cudaMemsetAsync(gmax, 0, (size_t)n_graphs * 4, a.stream);
    if (err != cudaSuccess) return err;
    err = cudaMemsetAsync(code, 0, (size_t)a.N * 2, a.stream);  // small graphs get no codes; the copy below reads them
    if (err != cudaSuccess) return err;
    const __nv_bfloat16* K = static_cast<const __nv_bfloat16*>(a.K);
    key_norm_kernel<<<(unsigned)((a.N * 32 + 255) / 256), 256, 0, a.stream>>>(K, (int)a.N, HD, a.graph_offsets, a.G, norm2,
                                                                             gmax, sb);
    const int DP = std::min(HD, kPivotDims);
    const int smem = (kPivots * (DP + 1) + kPivots) * 4;
    auto kern = pivot_code_kernel<true>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    kern<<<w.max_items, kAssignThreads, smem, a.stream>>>(K, K, HD, reinterpret_cast<const WorkItem*>(a.ws + w.items_off), sb,
                                                          a.graph_offsets, a.G, norm2, gmax, code);
    auto sort = graph_sort_stable_kernel<kKeyCodeBits2>;
    constexpr int sort_smem = (32 << kKeyCodeBits2) * 4;
    err = cudaFuncSetAttribute(sort, cudaFuncAttributeMaxDynamicSharedMemorySize, sort_smem);
    if (err != cudaSuccess) return err;
    sort<<<std::min(n_graphs, sm_count() * 2), kSortThreads, sort_smem, a.stream>>>(a.graph_offsets, a.G, (int)a.N, code, kperm, sb);
    const int vec_per_row = a.d * 2 / 16;
    const long long n_vec = (long long)a.N * a.H * vec_per_row;
    pack_keys_perm_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.K), kperm, reinterpret_cast<uint4*>(a.ws + w.kpack_off), n_vec, (int)a.N, a.H,
        vec_per_row, sb, code, code_sorted);
    return cudaGetLastError();
}

}  // namespace kmip
