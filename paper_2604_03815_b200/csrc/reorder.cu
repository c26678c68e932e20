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
#include <algorithm>

#include "common.cuh"

namespace kmip {

namespace {

constexpr int kCodeBits = 12;
constexpr int kBuckets = 1 << kCodeBits;
constexpr int kSortThreads = 1024;
constexpr int kMinRowsToSort = 8192;  // smaller graphs keep their order

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
__global__ void __launch_bounds__(kSortThreads)
graph_sort_kernel(const int32_t* __restrict__ offs, int G, int N, const unsigned short* __restrict__ code,
                  int* __restrict__ perm, const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;  // malformed offsets were reported by the plan kernel
    __shared__ int s_bin[kBuckets];
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
        // exclusive scan of the 4096 counts: four consecutive bins per thread
        int c[4], sum = 0;
#pragma unroll
        for (int x = 0; x < 4; ++x) { c[x] = s_bin[tid * 4 + x]; sum += c[x]; }
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
        for (int x = 0; x < 4; ++x) { s_bin[tid * 4 + x] = start; start += c[x]; }
        __syncthreads();
        for (int r = lo + tid; r < hi; r += kSortThreads) perm[atomicAdd(&s_bin[code[r]], 1)] = r;
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

}  // namespace

// After launch_plan (which validates the offsets): codes, per-graph bucket sort, permuted copy of Q.
cudaError_t launch_reorder_queries(const FwdArgs& a, const FwdWorkspace& w) {
    const StatusBlock* sb = reinterpret_cast<const StatusBlock*>(a.ws);
    unsigned short* code = reinterpret_cast<unsigned short*>(a.ws + w.code_off);
    int* perm = reinterpret_cast<int*>(a.ws + w.perm_off);
    const int HD = a.H * a.d;
    query_code_kernel<<<(unsigned)((a.N * 32 + 255) / 256), 256, 0, a.stream>>>(
        static_cast<const __nv_bfloat16*>(a.Q), (int)a.N, HD, code, sb);
    const int n_graphs = a.graph_offsets ? a.G : 1;
    graph_sort_kernel<<<std::min(n_graphs, 148 * 2), kSortThreads, 0, a.stream>>>(a.graph_offsets, a.G, (int)a.N, code, perm, sb);
    const int vec_per_row = HD * 2 / 16;
    const long long n_vec = (long long)a.N * vec_per_row;
    gather_rows_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.Q), perm, reinterpret_cast<uint4*>(a.ws + w.qperm_off), n_vec, vec_per_row, sb);
    return cudaGetLastError();
}

}  // namespace kmip
