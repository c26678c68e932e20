// Statistics for the pruned tensor-core sweep (not in the paper, which lists the quadratic search as
// its first limitation and rejects approximate indexes; this one is exact).
//
// A key tile T (128 consecutive keys of the sweep's key order, one head) can be left out for a block B
// of query rows when no key in it can reach the threshold tau_i of any row i of the block.  Two bounds
// on q_i . k_j over i in B, j in T are used, each from a few numbers per block and per tile:
//   centroid bound   with q_i = c_B + e_i, |e_i| <= r_B and k_j = c_T + f_j, |f_j| <= r_T:
//                    q_i . k_j <= c_B . c_T + |c_B| r_T + |c_T| r_B + r_B r_T;
//   norm bound       q_i . k_j <= |q_i| max_j |k_j|  (Cauchy-Schwarz), i.e. the tile is dead once
//                    max_j |k_j| < min_i tau_i / |q_i| over the rows with tau_i > 0.
// This file computes c, r, |c| and max |k| for every item's query rows and for every key tile, and the
// row norms |q_i|; the sweep's producer warp evaluates the bounds (score_select_tc.cu).  The key order
// (reorder.cu: heavy keys first, similar keys together) is what makes the tiles tight.
#include <algorithm>

#include "common.cuh"

namespace kmip {

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;

// Statistics of `n` rows of D bf16 values, row r at base + r * stride.  Record: c[0..D), r, |c|, max |row|, 0.
// The radius is taken against the stored fp32 centroid and rounded up, so the bounds hold for the
// numbers in the record whatever the rounding of the mean was.
template <int D>
__device__ void rows_stats(const __nv_bfloat16* __restrict__ base, size_t stride, int n, float* __restrict__ rec,
                           float* __restrict__ norms, int norm_stride) {
    constexpr int X = (D + 31) / 32;  // columns per lane
    __shared__ float s_sum[kWarps][D];
    __shared__ float s_c[D];
    __shared__ float s_red[2][kWarps];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    float acc[X], mx_norm2 = 0.0f;
#pragma unroll
    for (int x = 0; x < X; ++x) acc[x] = 0.0f;
    for (int r = wid; r < n; r += kWarps) {
        float s = 0.0f;
#pragma unroll
        for (int x = 0; x < X; ++x) {
            const int c = lane + 32 * x;
            const float v = c < D ? Elem<__nv_bfloat16>::load(base + (size_t)r * stride + c) : 0.0f;
            acc[x] += v;
            s = fmaf(v, v, s);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        mx_norm2 = fmaxf(mx_norm2, s);
        if (norms && lane == 0) norms[(size_t)r * norm_stride] = sqrtf(s);
    }
#pragma unroll
    for (int x = 0; x < X; ++x)
        if (lane + 32 * x < D) s_sum[wid][lane + 32 * x] = acc[x];
    __syncthreads();
    for (int c = threadIdx.x; c < D; c += kThreads) {
        float t = 0.0f;
        for (int w = 0; w < kWarps; ++w) t += s_sum[w][c];
        s_c[c] = t / (float)max(n, 1);
    }
    __syncthreads();
    float mx_dist2 = 0.0f;
    for (int r = wid; r < n; r += kWarps) {
        float s = 0.0f;
#pragma unroll
        for (int x = 0; x < X; ++x) {
            const int c = lane + 32 * x;
            if (c < D) {
                const float v = Elem<__nv_bfloat16>::load(base + (size_t)r * stride + c) - s_c[c];
                s = fmaf(v, v, s);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        mx_dist2 = fmaxf(mx_dist2, s);
    }
    if (lane == 0) { s_red[0][wid] = mx_dist2; s_red[1][wid] = mx_norm2; }
    __syncthreads();
    for (int c = threadIdx.x; c < D; c += kThreads) rec[c] = s_c[c];
    if (threadIdx.x == 0) {
        float d2 = 0.0f, n2 = 0.0f, c2 = 0.0f;
        for (int w = 0; w < kWarps; ++w) { d2 = fmaxf(d2, s_red[0][w]); n2 = fmaxf(n2, s_red[1][w]); }
        for (int c = 0; c < D; ++c) c2 = fmaf(s_c[c], s_c[c], c2);
        rec[D] = sqrtf(d2) * 1.0001f + 1e-30f;
        rec[D + 1] = sqrtf(c2) * 1.0001f;
        rec[D + 2] = sqrtf(n2) * 1.0001f;
        rec[D + 3] = 0.0f;
    }
    __syncthreads();  // the shared arrays are reused by the next call
}

// One block per (work item, head): the item's query tiles (sweep order) and the key tiles that start at
// the item's own row positions - an item covers rows_per_item = 128 * m rows of its graph from a multiple
// of 128 past the graph's first row, so all items of a graph together cover each of its key tiles once.
template <int D>
__global__ void __launch_bounds__(kThreads)
prune_stats_kernel(const __nv_bfloat16* __restrict__ Qs, const __nv_bfloat16* __restrict__ Kp,
                   const WorkItem* __restrict__ items, const StatusBlock* __restrict__ sb, int N, int H,
                   int rows_per_item, float* __restrict__ qnorm, float* __restrict__ qstat, float* __restrict__ kstat,
                   const unsigned short* __restrict__ qcode, const int* __restrict__ perm,
                   const unsigned short* __restrict__ kcode_sorted) {
    if (sb->status != KMIP_OK) return;
    const int item = blockIdx.x, h = blockIdx.y;
    if (item >= sb->n_items) return;
    const WorkItem it = items[item];
    constexpr int REC = D + 4;
    const int nqt = rows_per_item / 128;  // one record per 128-row query tile: the sweep skips (key tile, query tile) pairs
    for (int qt = 0; qt < nqt && qt * 128 < it.nrows; ++qt) {
        const int r0 = it.row0 + qt * 128;
        rows_stats<D>(Qs + ((size_t)r0 * H + h) * D, (size_t)H * D, min(128, it.nrows - qt * 128),
                      qstat + (((size_t)item * nqt + qt) * H + h) * REC, qnorm + (size_t)r0 * H + h, H);
    }
    if (threadIdx.x == 0) {
        // Start tile of the block's sweep: where the keys of the pivot its middle row scores highest against
        // begin (in the heaviest norm class, which is sorted first), so that the thresholds rise early.
        int jstart = 0;
        if (it.key_hi - it.key_lo >= kMinRowsToSort) {
            const unsigned target = qcode[perm[it.row0 + it.nrows / 2]];
            int a = it.key_lo, b = it.key_hi;  // first position whose code is >= target
            while (a < b) {
                const int m = (a + b) >> 1;
                if (kcode_sorted[m] < target) a = m + 1; else b = m;
            }
            jstart = a < it.key_hi ? (a - it.key_lo) / 128 : 0;
        }
        qstat[((size_t)item * nqt * H + h) * REC + D + 3] = __int_as_float(jstart);  // in the first tile's record
    }
    const int j_first = (it.row0 - it.key_lo) / 128;
    for (int t = 0; t < rows_per_item / 128; ++t) {
        const int p0 = it.row0 + t * 128;
        if (p0 >= it.key_hi) break;
        rows_stats<D>(Kp + ((size_t)h * N + p0) * D, (size_t)D, min(128, it.key_hi - p0),
                      kstat + ((size_t)(it.tile0 + j_first + t) * H + h) * REC, nullptr, 0);
    }
}

// One block per graph, one warp per head at a time: rec[D+3] of tile j becomes the largest key norm of the
// graph's tiles j, j+1, ... - once it is below every row's threshold / |q|, the rest of the graph is dead.
template <int D>
__global__ void __launch_bounds__(kThreads)
suffix_max_kernel(const int32_t* __restrict__ offs, int G, int N, int H, float* __restrict__ kstat,
                  const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    constexpr int REC = D + 4;
    const int g = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int lo = offs ? __ldg(offs + g) : 0, hi = offs ? __ldg(offs + g + 1) : N;
    const int ntiles = (hi - lo + 127) / 128, tile0 = lo / 128 + g;
    const int chunk = (ntiles + 31) / 32;
    for (int h = wid; h < H; h += kWarps) {
        const int j_lo = min(ntiles, lane * chunk), j_hi = min(ntiles, j_lo + chunk);
        float m = 0.0f;
        for (int j = j_lo; j < j_hi; ++j) m = fmaxf(m, kstat[((size_t)(tile0 + j) * H + h) * REC + D + 2]);
        // largest norm of all later lanes' chunks
        float later = 0.0f;
#pragma unroll
        for (int l = 1; l < 32; ++l) {
            const float t = __shfl_sync(0xFFFFFFFFu, m, l);
            if (l > lane) later = fmaxf(later, t);
        }
        float run = later;
        for (int j = j_hi - 1; j >= j_lo; --j) {
            float* rec = kstat + ((size_t)(tile0 + j) * H + h) * REC;
            run = fmaxf(run, rec[D + 2]);
            rec[D + 3] = run;
        }
    }
}

template <int D>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w) {
    const dim3 grid((unsigned)w.max_items, (unsigned)a.H);
    prune_stats_kernel<D><<<grid, kThreads, 0, a.stream>>>(
        reinterpret_cast<const __nv_bfloat16*>(a.ws + w.qperm_off), reinterpret_cast<const __nv_bfloat16*>(a.ws + w.kpack_off),
        reinterpret_cast<const WorkItem*>(a.ws + w.items_off), reinterpret_cast<const StatusBlock*>(a.ws), (int)a.N, a.H,
        score_select_tc_rows_per_item(a.d, a.k), reinterpret_cast<float*>(a.ws + w.qnorm_off),
        reinterpret_cast<float*>(a.ws + w.qstat_off), reinterpret_cast<float*>(a.ws + w.kstat_off),
        reinterpret_cast<const unsigned short*>(a.ws + w.code_off), reinterpret_cast<const int*>(a.ws + w.perm_off),
        reinterpret_cast<const unsigned short*>(a.ws + w.kcs_off));
    const int n_graphs = a.graph_offsets ? a.G : 1;
    suffix_max_kernel<D><<<n_graphs, kThreads, 0, a.stream>>>(a.graph_offsets, a.G, (int)a.N, a.H,
                                                             reinterpret_cast<float*>(a.ws + w.kstat_off),
                                                             reinterpret_cast<const StatusBlock*>(a.ws));
    return cudaGetLastError();
}

}  // namespace

// After launch_reorder_queries and launch_reorder_keys (reads the sweep-order copies of Q and K).
cudaError_t launch_prune_stats(const FwdArgs& a, const FwdWorkspace& w) {
    switch (a.d) {
        case 16: return launch_d<16>(a, w);
        case 32: return launch_d<32>(a, w);
        case 64: return launch_d<64>(a, w);
        case 128: return launch_d<128>(a, w);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace kmip
