// CUDA-core score + running top-k kernel for KMIP_FP32_EXACT with k <= 32 and d <= 64
// (Algorithm 1 lines 2-3), tiled: one thread per query row, keys staged in shared memory.
//
// Every score is d fused multiply-adds in fp32 in index order c = 0..d-1, exactly as in
// score_select_exact.cu, but a key tile is read from global memory once per 128 query rows
// instead of once per row: a block owns 128 rows of one graph and one head, keeps each row's q in
// registers, streams the graph's keys through a double-buffered shared-memory tile
// (cp.async) and every thread walks the tile, eight keys (one group) at a time, with
// broadcast reads.  As in the tensor-core sweep the candidates are 8-key groups ranked by
// (maximum desc, first key asc): the k best groups always contain the k best keys under
// (score desc, key asc), ties included, because the lists compare the full 64-bit
// (score, ~key) words here.  refine.cu rescores the 8k keys of a row and keeps the best k.
#include <algorithm>

#include "common.cuh"
#include "topk_buffer.cuh"

namespace kmip {

namespace {

constexpr int ROWS = 128;  // query rows per block = threads per block
constexpr int TK = 64;     // keys per shared-memory tile
constexpr int GK = 8;      // keys per candidate group
constexpr int LIST = 32;   // list slots per row (k <= LIST)
constexpr int KG = LIST / 8;
constexpr int ROOM = 16;   // pending slots per row; a tile adds at most TK / GK = 8

// Per-row state of one thread.  The row's list and pending slots live in shared memory in
// slot-major order (slot s of thread t at [s * ROWS + t]): no bank conflicts, whatever the
// threads of a warp do.  gmin caches the minimum of each 8-slot block, lmin that of the list
// (0 = empty slot, so tau stays -inf until k groups are in).
struct RowState {
    cand_t gmin[KG];
    cand_t lmin;
    float tau;
    int cnt;
};

__device__ __forceinline__ void flush_row(RowState& r, cand_t* list, const cand_t* pend, bool rvalid) {
    for (int t = 0; t < r.cnt; ++t) {
        const cand_t x = pend[t * ROWS];
        if (x > r.lmin) {
            int g = 0;
            cand_t m = r.gmin[0];
#pragma unroll
            for (int q = 1; q < KG; ++q)
                if (r.gmin[q] < m) { m = r.gmin[q]; g = q; }
            cand_t* grp = list + (g * 8) * ROWS;
            cand_t nm = x;
            int pos = -1;
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const cand_t y = grp[s * ROWS];
                if (y == m && pos < 0) pos = s; else nm = cmin(nm, y);
            }
            grp[pos * ROWS] = x;
#pragma unroll
            for (int q = 0; q < KG; ++q)
                if (q == g) r.gmin[q] = nm;
            cand_t lm = r.gmin[0];
#pragma unroll
            for (int q = 1; q < KG; ++q) lm = cmin(lm, r.gmin[q]);
            r.lmin = lm;
        }
    }
    r.cnt = 0;
    if (rvalid) r.tau = r.lmin ? cand_score(r.lmin) : -CUDART_INF_F;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Copies keys [key0, key0 + n) of head h (n <= TK rows of D floats, row stride H*D) into a tile.
template <int D>
__device__ __forceinline__ void load_key_tile(float* tile, const float* __restrict__ K, int key0, int n, int h, int H) {
    constexpr int V = D / 4;  // 16-byte pieces per key
    for (int x = threadIdx.x; x < n * V; x += ROWS) {
        const int r = x / V, v = x % V;
        cp_async16(tile + r * D + v * 4, K + ((size_t)(key0 + r) * H + h) * D + v * 4);
    }
}

template <int D>
__global__ void __launch_bounds__(ROWS)
score_select_fp32_kernel(const float* __restrict__ Q, const float* __restrict__ K, const WorkItem* __restrict__ items,
                         const StatusBlock* __restrict__ sb, int H, int k, int32_t* __restrict__ topk_idx,
                         float* __restrict__ topk_score) {
    if (sb->status != KMIP_OK) return;  // the plan kernel rejected the offsets
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sK = reinterpret_cast<float*>(smem_raw);                                // [2][TK][D]
    cand_t* sList = reinterpret_cast<cand_t*>(smem_raw + 2 * TK * D * sizeof(float));  // [LIST][ROWS]
    cand_t* sPend = sList + LIST * ROWS;                                            // [ROOM][ROWS]
    const int tid = threadIdx.x;
    cand_t* list = sList + tid;
    cand_t* pend = sPend + tid;

    const int n_items = sb->n_items;
    const long long total = (long long)n_items * H;
    for (long long w = blockIdx.x; w < total; w += gridDim.x) {
        const int h = (int)(w / n_items);
        const WorkItem it = items[w % n_items];
        const bool rvalid = tid < it.nrows;
        const int row = it.row0 + (rvalid ? tid : 0);

        float q[D];
#pragma unroll
        for (int c = 0; c < D; c += 4) {
            const float4 t = *reinterpret_cast<const float4*>(Q + ((size_t)row * H + h) * D + c);
            q[c] = t.x; q[c + 1] = t.y; q[c + 2] = t.z; q[c + 3] = t.w;
        }
        RowState rs;
        for (int s = 0; s < LIST; ++s) list[s * ROWS] = (s < k) ? 0ull : ~0ull;  // slots past k are never the minimum
#pragma unroll
        for (int g = 0; g < KG; ++g) rs.gmin[g] = (8 * g < k) ? 0ull : ~0ull;
        rs.lmin = 0ull;
        rs.tau = rvalid ? -CUDART_INF_F : CUDART_INF_F;
        rs.cnt = 0;

        const int ntiles = (it.key_hi - it.key_lo + TK - 1) / TK;
        __syncthreads();  // the previous item's readers are done with the key tiles
        load_key_tile<D>(sK, K, it.key_lo, min(TK, it.key_hi - it.key_lo), h, H);
        for (int t = 0; t < ntiles; ++t) {
            cp_async_wait_all();
            __syncthreads();  // tile t has landed; everybody is done with tile t-1
            const int key0 = it.key_lo + t * TK;
            if (t + 1 < ntiles)
                load_key_tile<D>(sK + ((t + 1) & 1) * TK * D, K, key0 + TK, min(TK, it.key_hi - key0 - TK), h, H);
            const float* tile = sK + (t & 1) * TK * D;
            const int nvalid = it.key_hi - key0;  // below TK only in the last tile
#pragma unroll 1
            for (int g = 0; g < TK / GK; ++g) {
                if (g * GK >= nvalid) break;
                float acc[GK];
#pragma unroll
                for (int j = 0; j < GK; ++j) acc[j] = 0.0f;
                const float* kg = tile + g * GK * D;
#pragma unroll
                for (int c = 0; c < D; c += 4) {
#pragma unroll
                    for (int j = 0; j < GK; ++j) {
                        const float4 kv = *reinterpret_cast<const float4*>(kg + j * D + c);  // same address in every thread
                        acc[j] = fmaf(q[c], kv.x, acc[j]);
                        acc[j] = fmaf(q[c + 1], kv.y, acc[j]);
                        acc[j] = fmaf(q[c + 2], kv.z, acc[j]);
                        acc[j] = fmaf(q[c + 3], kv.w, acc[j]);
                    }
                }
                if (g * GK + GK > nvalid) {  // keys past the end of the graph do not exist
#pragma unroll
                    for (int j = 0; j < GK; ++j)
                        if (g * GK + j >= nvalid) acc[j] = -CUDART_INF_F;
                }
                const float gmax = fmaxf(fmaxf(fmaxf(acc[0], acc[1]), fmaxf(acc[2], acc[3])),
                                         fmaxf(fmaxf(acc[4], acc[5]), fmaxf(acc[6], acc[7])));
                if (gmax > rs.tau) {
                    pend[rs.cnt * ROWS] = make_cand(gmax, key0 + g * GK);
                    ++rs.cnt;
                }
            }
            // a tile adds at most 8 groups per row
            if (__any_sync(0xFFFFFFFFu, rs.cnt > ROOM - TK / GK)) flush_row(rs, list, pend, rvalid);
        }
        flush_row(rs, list, pend, rvalid);
        if (rvalid) {
            // the row's k groups (first key, group maximum), unsorted; empty slots as -1 / -inf
            const size_t o = ((size_t)row * H + h) * k;
            for (int s = 0; s < k; ++s) {
                const cand_t c = list[s * ROWS];
                topk_idx[o + s] = c ? cand_index(c) : -1;
                topk_score[o + s] = c ? cand_score(c) : -CUDART_INF_F;
            }
        }
    }
}

template <int D>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w) {
    constexpr size_t smem = 2 * TK * D * sizeof(float) + (size_t)(LIST + ROOM) * ROWS * sizeof(cand_t);
    auto kern = score_select_fp32_kernel<D>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    const long long total = (long long)w.max_items * a.H;
    const int grid = (int)std::min<long long>(total, (long long)sm_count() * 16);
    kern<<<grid, ROWS, smem, a.stream>>>(static_cast<const float*>(a.Q), static_cast<const float*>(a.K),
                                         reinterpret_cast<const WorkItem*>(a.ws + w.items_off),
                                         reinterpret_cast<const StatusBlock*>(a.ws), a.H, a.k, a.topk_idx, a.topk_score);
    return cudaGetLastError();
}

}  // namespace

bool score_select_fp32_tiled_supported(int32_t d, int32_t k) { return (d == 16 || d == 32 || d == 64) && k <= LIST; }

cudaError_t launch_score_select_fp32_tiled(const FwdArgs& a, const FwdWorkspace& w) {
    switch (a.d) {
        case 16: return launch_d<16>(a, w);
        case 32: return launch_d<32>(a, w);
        case 64: return launch_d<64>(a, w);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace kmip
