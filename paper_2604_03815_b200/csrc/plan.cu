// Plan kernel: CSR graph offsets -> work items of the tensor-core score kernel.
// The paper leaves open how the graphs of a batch are kept apart; here a query only ever sees
// the key range of its own graph, so each item carries that range.  Runs on the device so the
// host never reads graph_offsets.
#include "common.cuh"

namespace kmip {

namespace {

constexpr int kPlanThreads = 1024;

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t* __restrict__ offs, int G, int N, int rows_per_item, int max_items,
            WorkItem* __restrict__ items, StatusBlock* __restrict__ sb) {
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    __shared__ int s_bad;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) { s_carry = 0; s_bad = 0; }
    __syncthreads();

    if (offs != nullptr) {
        int bad = 0;
        if (tid == 0 && (__ldg(offs) != 0 || __ldg(offs + G) != N)) bad = 1;
        for (int g = tid; g < G; g += kPlanThreads)
            if (__ldg(offs + g) > __ldg(offs + g + 1) || __ldg(offs + g) < 0) bad = 1;
        if (bad) s_bad = 1;
        __syncthreads();
        if (s_bad) {
            if (tid == 0) { record_status(sb, KMIP_ERR_BAD_OFFSETS, 1); sb->n_items = 0; }
            return;
        }
    }

    const int n_graphs = offs ? G : 1;
    for (int g0 = 0; g0 < n_graphs; g0 += kPlanThreads) {
        const int g = g0 + tid;
        int lo = 0, hi = 0;
        if (g < n_graphs) {
            lo = offs ? __ldg(offs + g) : 0;
            hi = offs ? __ldg(offs + g + 1) : N;
        }
        const int tiles = (hi - lo + rows_per_item - 1) / rows_per_item;
        // block-wide exclusive scan of `tiles`
        int incl = tiles;
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
            s_warp[lane] = w;  // inclusive over warps
        }
        __syncthreads();
        const int base = s_carry + (wid ? s_warp[wid - 1] : 0) + incl - tiles;
        for (int t = 0; t < tiles; ++t) {
            if (base + t < max_items) {
                WorkItem it;
                it.row0 = lo + t * rows_per_item;
                it.nrows = min(rows_per_item, hi - it.row0);
                it.key_lo = lo;
                it.key_hi = hi;
                it.tile0 = lo / 128 + g;
                items[base + t] = it;
            }
        }
        __syncthreads();
        if (tid == 0) s_carry += s_warp[31];
        __syncthreads();
    }
    if (tid == 0) sb->n_items = min(s_carry, max_items);
}

// K [N, H, d] -> [H, N, d], 16 bytes per thread.
__global__ void pack_keys_kernel(const uint4* __restrict__ K, uint4* __restrict__ Kp, long long n_vec, int N, int H,
                                 int vec_per_row) {
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const long long rowh = v / vec_per_row;  // j * H + h
    const int c = (int)(v % vec_per_row);
    const long long j = rowh / H;
    const int h = (int)(rowh % H);
    Kp[((long long)h * N + j) * vec_per_row + c] = __ldg(K + v);
}

__global__ void canary_kernel(unsigned char* __restrict__ ws, const Canaries c, bool fill) {
    const int blk = blockIdx.x;
    if (blk >= c.n) return;
    uint32_t* p = reinterpret_cast<uint32_t*>(ws + c.off[blk]);
    StatusBlock* sb = reinterpret_cast<StatusBlock*>(ws);
    for (int i = threadIdx.x; i < (int)(kCanaryBytes / 4); i += blockDim.x) {
        if (fill) p[i] = kCanaryWord;
        else if (p[i] != kCanaryWord) record_status(sb, KMIP_ERR_CHECK, 900 + blk);
    }
}

}  // namespace

cudaError_t launch_canary_fill(unsigned char* ws, const Canaries& c, cudaStream_t stream) {
    if (!kChecks || c.n == 0) return cudaSuccess;
    canary_kernel<<<c.n, 64, 0, stream>>>(ws, c, true);
    return cudaGetLastError();
}

cudaError_t launch_canary_check(unsigned char* ws, const Canaries& c, cudaStream_t stream) {
    if (!kChecks || c.n == 0) return cudaSuccess;
    canary_kernel<<<c.n, 64, 0, stream>>>(ws, c, false);
    return cudaGetLastError();
}

cudaError_t launch_pack_keys(const FwdArgs& a, const FwdWorkspace& w) {
    const int vec_per_row = a.d * 2 / 16;
    const long long n_vec = (long long)a.N * a.H * vec_per_row;
    pack_keys_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.K), reinterpret_cast<uint4*>(a.ws + w.kpack_off), n_vec, (int)a.N, a.H, vec_per_row);
    return cudaGetLastError();
}

cudaError_t launch_plan(const FwdArgs& a, const FwdWorkspace& w, int rows_per_item) {
    plan_kernel<<<1, kPlanThreads, 0, a.stream>>>(
        a.graph_offsets, a.G, (int)a.N, rows_per_item, w.max_items,
        reinterpret_cast<WorkItem*>(a.ws + w.items_off), reinterpret_cast<StatusBlock*>(a.ws));
    return cudaGetLastError();
}

}  // namespace kmip
