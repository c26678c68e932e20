// Tensor-core score + running top-k kernel (Algorithm 1 lines 2-3) for sm_100a.
//
// The paper evaluates S = Q K^T lazily (a "symbolic matrix") on CUDA cores and reduces each row
// to its k best entries without storing S.  Here the same reduction is fed by the 5th-generation
// tensor cores: a persistent CTA per SM owns up to 256 query rows (two 128-row tiles) of one
// graph and one head, streams that graph's keys in 128-key tiles through a TMA -> shared memory
// ring, multiplies each tile against both query tiles with tcgen05.mma (bf16 in, fp32
// accumulators in tensor memory, double buffered), and eight selection warps read the
// accumulators straight out of tensor memory.  One thread owns one query row: it reduces 32
// scores to their maximum with three-input max instructions, compares once against the row's
// threshold, and only on a hit rescans and appends candidates to the row's buffer in shared
// memory (topk_buffer.cuh).  The N x N scores never leave the SM.
//
// Warp roles (NQT = query tiles per CTA, 1 or 2):
//   warps 0 .. 4*NQT-1   selection; warp w reads TMEM lanes 32*(w%4).. of query tile w/4
//   warp 4*NQT           TMA producer (one lane)
//   warp 4*NQT+1         TMEM allocation + tcgen05.mma issue (one lane)
// Every wait is bounded; on expiry the CTA records KMIP_ERR_TIMEOUT, drains and exits normally.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"
#include "topk_buffer.cuh"

namespace kmip {

namespace {

constexpr int BM = 128;  // query rows per tile = TMEM lanes
constexpr int BN = 128;  // keys per tile = accumulator columns
constexpr unsigned FULL = 0xFFFFFFFFu;

template <int D>
struct TcShape {
    static constexpr int RB = D * 2;                        // bytes per operand row
    static constexpr int SWB = RB >= 128 ? 128 : RB;        // swizzle span = shared-memory row pitch
    static constexpr int KCH = RB / SWB;                    // 128-byte column chunks per row
    static constexpr int BOX_INNER = SWB / 2;               // elements per TMA box row
    static constexpr uint32_t LAYOUT = SWB == 128 ? 2u : (SWB == 64 ? 4u : 6u);  // UMMA swizzle code
    static constexpr int KSTEPS = D / 16;                   // one tcgen05.mma covers 16 bf16 of depth
    static constexpr int STEPS_PER_CH = SWB / 32;
    static constexpr int CH_BYTES = 128 * SWB;              // one chunk of a 128-row tile
    static constexpr int TILE_BYTES = 128 * RB;
};

// Shared-memory matrix descriptor of a K-major, swizzled operand whose 8-row groups are
// contiguous (stride = 8 * pitch).  The leading-dimension field is unused for this layout.
template <int D>
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    using Sh = TcShape<D>;
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((8 * Sh::SWB) >> 4) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of sm_100
    d |= (uint64_t)Sh::LAYOUT << 61;
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128, N = BN.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                ((uint32_t)(BM >> 4) << 24);

template <int E, int NQT, int S>
struct SmemPlan {
    static constexpr int CAP = 32 * E;
    static constexpr int ROW_STRIDE = CAP + 1;  // odd pitch: simultaneous appends hit distinct banks
    static constexpr int NBARS = 3 + 2 * S + 4 * NQT;
};

struct Bars {
    uint32_t base;
    int S, NQT;
    __device__ uint32_t q_full() const { return base; }
    __device__ uint32_t q_empty() const { return base + 8; }
    __device__ uint32_t done() const { return base + 16; }
    __device__ uint32_t k_full(int s) const { return base + 8 * (3 + s); }
    __device__ uint32_t k_empty(int s) const { return base + 8 * (3 + S + s); }
    __device__ uint32_t t_full(int qt, int b) const { return base + 8 * (3 + 2 * S + qt * 2 + b); }
    __device__ uint32_t t_empty(int qt, int b) const { return base + 8 * (3 + 2 * S + 2 * NQT + qt * 2 + b); }
};

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              StatusBlock* sb, int who) {
    if (ptx::mbar_wait_bounded(bar, parity, abort_flag)) return true;
    record_status(sb, KMIP_ERR_TIMEOUT, who);
    return false;
}

// Threshold test and candidate append for 32 consecutive scores of this thread's row.
// Warp-uniform control flow: the rescan and the compactions are entered by all 32 lanes.
template <int E>
__device__ __forceinline__ void filter_chunk(const uint32_t (&v)[32], int key0, int nvalid, float& tau, int& cnt,
                                             cand_t* myrow, cand_t* wrows, int k, int lane) {
    constexpr int CAP = 32 * E;
    constexpr int RS = CAP + 1;
    float f[32];
#pragma unroll
    for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
    if (nvalid < 32) {  // ragged end of the graph's key range: columns past it do not exist
#pragma unroll
        for (int x = 0; x < 32; ++x)
            if (x >= nvalid) f[x] = -CUDART_INF_F;
    }
    float sub[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        float m = ptx::max3(f[8 * g], f[8 * g + 1], f[8 * g + 2]);
        m = ptx::max3(m, f[8 * g + 3], f[8 * g + 4]);
        m = ptx::max3(m, f[8 * g + 5], f[8 * g + 6]);
        sub[g] = fmaxf(m, f[8 * g + 7]);
    }
    const float gm = fmaxf(ptx::max3(sub[0], sub[1], sub[2]), sub[3]);
    if (__any_sync(FULL, gm > tau)) {
        const int room = CAP - k;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            if (__any_sync(FULL, sub[g] > tau)) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int x = 8 * g + c;
                    if (f[x] > tau) {
                        myrow[k + cnt] = make_cand(f[x], key0 + x);
                        ++cnt;
                    }
                }
                unsigned need = __ballot_sync(FULL, cnt > room - 8);
                while (need) {
                    const int r = __ffs(need) - 1;
                    need &= need - 1;
                    const int rc = __shfl_sync(FULL, cnt, r);
                    const float nt = warp_compact_row<E>(wrows + r * RS, k, rc, lane);
                    if (lane == r) {
                        tau = nt;
                        cnt = 0;
                    }
                }
            }
        }
    }
}

template <int D, int E, int NQT, int S, bool DUMP>
__global__ void __launch_bounds__(NQT * 128 + 64, 1)
score_select_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const WorkItem* __restrict__ items, StatusBlock* __restrict__ sb, int H, int k,
                       int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                       float* __restrict__ dump, int dump_ld) {
    using Sh = TcShape<D>;
    using Sp = SmemPlan<E, NQT, S>;
    constexpr int CAP = Sp::CAP, RS = Sp::ROW_STRIDE;
    constexpr int NEPI = 4 * NQT;
    constexpr uint32_t TMEM_COLS = NQT * 2 * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + NQT * Sh::TILE_BYTES;
    cand_t* sRows = reinterpret_cast<cand_t*>(sK + S * Sh::TILE_BYTES);
    uint64_t* sBars = reinterpret_cast<uint64_t*>(sRows + NQT * 128 * RS);
    uint32_t* sTmem = reinterpret_cast<uint32_t*>(sBars + Sp::NBARS);
    volatile int* sAbort = reinterpret_cast<volatile int*>(sTmem + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Bars bars{ptx::smem_u32(sBars), S, NQT};

    if (threadIdx.x == 0) {
        ptx::mbar_init(bars.q_full(), 1);
        ptx::mbar_init(bars.q_empty(), 1);
        ptx::mbar_init(bars.done(), 1);
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(bars.k_full(s), 1);
            ptx::mbar_init(bars.k_empty(s), 1);
        }
        for (int qt = 0; qt < NQT; ++qt)
            for (int b = 0; b < 2; ++b) {
                ptx::mbar_init(bars.t_full(qt, b), 1);
                ptx::mbar_init(bars.t_empty(qt, b), 4);  // one arrival per selection warp of the tile
            }
        *sAbort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == NEPI + 1) {
        ptx::tmem_alloc(ptx::smem_u32(sTmem), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    if (warp == NEPI && lane == 0) {
        ptx::prefetch_tensormap(&tmQ);
        ptx::prefetch_tensormap(&tmK);
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *sTmem;

    const int n_items = sb->n_items;
    const long long total = (long long)n_items * H;

    if (warp == NEPI) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int kt = 0, ic = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
                const int h = (int)(w / n_items);
                const WorkItem it = items[w % n_items];
                if (!(ok = wait_or_abort(bars.q_empty(), (ic & 1) ^ 1, sAbort, sb, 1))) break;
                ptx::mbar_arrive_expect_tx(bars.q_full(), NQT * Sh::TILE_BYTES);
                for (int qt = 0; qt < NQT; ++qt)
                    for (int ch = 0; ch < Sh::KCH; ++ch)
                        ptx::tma_load_2d(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmQ,
                                         h * D + ch * 64, it.row0 + qt * BM, bars.q_full());
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; j < ntiles; ++j, ++kt) {
                    const int s = kt % S;
                    if (!(ok = wait_or_abort(bars.k_empty(s), ((kt / S) & 1) ^ 1, sAbort, sb, 2))) break;
                    ptx::mbar_arrive_expect_tx(bars.k_full(s), Sh::TILE_BYTES);
                    for (int ch = 0; ch < Sh::KCH; ++ch)
                        ptx::tma_load_2d(ptx::smem_u32(sK + s * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmK,
                                         h * D + ch * 64, it.key_lo + j * BN, bars.k_full(s));
                }
                ++ic;
            }
            if (!ok) {
                // give copies that are still in flight a bounded time to land before the CTA exits
                const uint64_t t0 = ptx::globaltimer_ns();
                for (int s = 0; s < S && kt > 0; ++s) {
                    const int last = kt - 1 - ((kt - 1 - s) % S + S) % S;  // last tile issued into stage s
                    if (last < 0) continue;
                    while (!ptx::mbar_try_wait(bars.k_full(s), (last / S) & 1) &&
                           ptx::globaltimer_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == NEPI + 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int kt = 0, ic = 0;
            int tc[2] = {0, 0};
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
                const WorkItem it = items[w % n_items];
                const int nq = (NQT == 2 && it.nrows > BM) ? 2 : 1;
                if (!(ok = wait_or_abort(bars.q_full(), ic & 1, sAbort, sb, 3))) break;
                ptx::tc_fence_after();
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; ok && j < ntiles; ++j, ++kt) {
                    const int s = kt % S;
                    if (!(ok = wait_or_abort(bars.k_full(s), (kt / S) & 1, sAbort, sb, 4))) break;
                    ptx::tc_fence_after();
                    for (int qt = 0; qt < nq; ++qt) {
                        const int b = tc[qt] & 1;
                        if (!(ok = wait_or_abort(bars.t_empty(qt, b), ((tc[qt] >> 1) & 1) ^ 1, sAbort, sb, 5))) break;
                        ptx::tc_fence_after();
                        const uint32_t d_tmem = tmem_base + (uint32_t)((qt * 2 + b) * BN);
#pragma unroll
                        for (int ks = 0; ks < Sh::KSTEPS; ++ks) {
                            const int off = (ks / Sh::STEPS_PER_CH) * Sh::CH_BYTES + (ks % Sh::STEPS_PER_CH) * 32;
                            const uint64_t da = make_smem_desc<D>(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + off));
                            const uint64_t db = make_smem_desc<D>(ptx::smem_u32(sK + s * Sh::TILE_BYTES + off));
                            ptx::mma_bf16_ss(d_tmem, da, db, kInstrDesc, ks > 0 ? 1u : 0u);
                        }
                        ptx::mma_commit(bars.t_full(qt, b));
                        ++tc[qt];
                    }
                    if (!ok) break;
                    ptx::mma_commit(bars.k_empty(s));
                }
                if (!ok) break;
                ptx::mma_commit(bars.q_empty());
                ++ic;
            }
            // all issued MMAs must have retired before tensor memory is released
            ptx::mma_commit(bars.done());
            const uint64_t t0 = ptx::globaltimer_ns();
            while (!ptx::mbar_try_wait(bars.done(), 0) && ptx::globaltimer_ns() - t0 < 1000000000ull) {}
        }
    } else {
        // ------------------------------------------------------------------ selection warps
        const int qt = warp >> 2, quarter = warp & 3;
        cand_t* wrows = sRows + (qt * 128 + quarter * 32) * RS;
        cand_t* myrow = wrows + lane * RS;
        int tcnt = 0;
        bool ok = true;
        for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
            const int h = (int)(w / n_items);
            const WorkItem it = items[w % n_items];
            if (qt * BM >= it.nrows) continue;  // this query tile is empty for the item
            const int local = qt * BM + quarter * 32 + lane;
            const bool rvalid = local < it.nrows;
            for (int t = 0; t < k; ++t) myrow[t] = 0ull;
            float tau = rvalid ? -CUDART_INF_F : CUDART_INF_F;
            int cnt = 0;
            __syncwarp();
            const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
            for (int j = 0; j < ntiles; ++j, ++tcnt) {
                const int b = tcnt & 1;
                ok = wait_or_abort(bars.t_full(qt, b), (tcnt >> 1) & 1, sAbort, sb, 6);
                ok = __all_sync(FULL, ok);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((qt * 2 + b) * BN);
                const int key0 = it.key_lo + j * BN;
                const int ncol = min(BN, it.key_hi - key0);
                uint32_t va[32], vb[32];
                ptx::tmem_ld_32x32(taddr, va);
#pragma unroll
                for (int c = 0; c < BN / 32; c += 2) {
                    ptx::tmem_ld_wait(va);
                    ptx::tmem_ld_32x32(taddr + (c + 1) * 32, vb);
                    if (DUMP) {
                        if (rvalid)
                            for (int x = 0; x < 32; ++x)
                                if (c * 32 + x < ncol)
                                    dump[((size_t)h * dump_ld + it.row0 + local) * dump_ld + key0 + c * 32 + x] = __uint_as_float(va[x]);
                    } else {
                        filter_chunk<E>(va, key0 + c * 32, ncol - c * 32, tau, cnt, myrow, wrows, k, lane);
                    }
                    ptx::tmem_ld_wait(vb);
                    if (c + 2 < BN / 32) ptx::tmem_ld_32x32(taddr + (c + 2) * 32, va);
                    if (DUMP) {
                        if (rvalid)
                            for (int x = 0; x < 32; ++x)
                                if ((c + 1) * 32 + x < ncol)
                                    dump[((size_t)h * dump_ld + it.row0 + local) * dump_ld + key0 + (c + 1) * 32 + x] = __uint_as_float(vb[x]);
                    } else {
                        filter_chunk<E>(vb, key0 + (c + 1) * 32, ncol - (c + 1) * 32, tau, cnt, myrow, wrows, k, lane);
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bars.t_empty(qt, b));
            }
            if (!ok) break;
            if (!DUMP) {
                // finalise: one last compaction per row leaves the sorted best k in slots [0,k)
                const int nloc = min(32, it.nrows - (qt * BM + quarter * 32));
                for (int r = 0; r < nloc; ++r) {
                    const int rc = __shfl_sync(FULL, cnt, r);
                    warp_compact_row<E>(wrows + r * RS, k, rc, lane);
                    const size_t o = ((size_t)(it.row0 + qt * BM + quarter * 32 + r) * H + h) * k;
                    warp_store_row(wrows + r * RS, k, lane, topk_idx + o, topk_score + o);
                }
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == NEPI + 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map over one [N, H*d] bf16 array; a box is 128 rows x one swizzle span of columns.
template <int D>
bool make_tensor_map(CUtensorMap* tm, const void* base, int64_t N, int H) {
    using Sh = TcShape<D>;
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)H * D, (cuuint64_t)N};
    const cuuint64_t gstride[1] = {(cuuint64_t)H * D * 2};
    const cuuint32_t box[2] = {(cuuint32_t)Sh::BOX_INNER, 128u};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUtensorMapSwizzle sw = Sh::SWB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : Sh::SWB == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int sms[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (sms[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        sms[dev] = v;
    }
    return sms[dev];
}

template <int D, int E, int NQT, int S, bool DUMP>
cudaError_t launch_cfg(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    using Sh = TcShape<D>;
    using Sp = SmemPlan<E, NQT, S>;
    constexpr size_t smem_bytes = 1024 + (size_t)(NQT + S) * Sh::TILE_BYTES + (size_t)NQT * 128 * Sp::ROW_STRIDE * 8 +
                                  (size_t)Sp::NBARS * 8 + 16;
    static_assert(smem_bytes <= 232448, "shared memory budget of one CTA");
    CUtensorMap tmQ, tmK;
    if (!make_tensor_map<D>(&tmQ, a.Q, a.N, a.H) || !make_tensor_map<D>(&tmK, a.K, a.N, a.H))
        return cudaErrorInvalidValue;
    auto kern = score_select_tc_kernel<D, E, NQT, S, DUMP>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (err != cudaSuccess) return err;
    const long long max_total = (long long)w.max_items * a.H;
    const int grid = (int)std::min<long long>(sm_count(), max_total);
    kern<<<grid, NQT * 128 + 64, smem_bytes, a.stream>>>(
        tmQ, tmK, reinterpret_cast<const WorkItem*>(a.ws + w.items_off), reinterpret_cast<StatusBlock*>(a.ws),
        a.H, a.k, a.topk_idx, a.topk_score, dump, (int)a.N);
    return cudaGetLastError();
}

template <int D, bool DUMP>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    constexpr int S = D <= 32 ? 4 : 3;
    if constexpr (D <= 64) {
        if (a.k <= 32) return launch_cfg<D, 2, 2, S, DUMP>(a, w, dump);
        return launch_cfg<D, 4, 1, S, DUMP>(a, w, dump);
    } else {
        if (a.k <= 32) return launch_cfg<D, 2, 1, S, DUMP>(a, w, dump);
        return cudaErrorNotSupported;
    }
}

template <bool DUMP>
cudaError_t launch_any(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    switch (a.d) {
        case 16: return launch_d<16, DUMP>(a, w, dump);
        case 32: return launch_d<32, DUMP>(a, w, dump);
        case 64: return launch_d<64, DUMP>(a, w, dump);
        case 128: return launch_d<128, DUMP>(a, w, dump);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace

bool score_select_tc_supported(int32_t d, int32_t k) {
    if (d != 16 && d != 32 && d != 64 && d != 128) return false;
    if (k <= 32) return true;
    return k <= 96 && d <= 64;
}

int score_select_tc_rows_per_item(int32_t d, int32_t k) { return (k <= 32 && d <= 64) ? 256 : 128; }

cudaError_t launch_score_select_tc(const FwdArgs& a, const FwdWorkspace& w) {
    return launch_any<false>(a, w, nullptr);
}

// Test hook: same TMA / tcgen05 pipeline, but the selection warps write every score of the tile to
// dump[h][i][j] (ld = N) instead of filtering.  Only for small single problems.
cudaError_t launch_score_dump_tc(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    return launch_any<true>(a, w, dump);
}

}  // namespace kmip
