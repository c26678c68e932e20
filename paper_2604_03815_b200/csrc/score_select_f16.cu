// Half-precision prefilter sweep of the tensor-core mode (Algorithm 1 lines 2-3) for head widths
// 16 and 32 and 16 < k <= 32 (k <= 16: score_select_f16x4.cu, the same filter on another pipeline).
//
// The paper lists half-precision arithmetic and tensor-core support as the engineering it left open
// (Sec. 6; closing remark of the FlashAttention comparison in the appendix).  The sweep of
// score_select_tc.cu is bound by the instructions that reduce the fp32 scores to group maxima, not by
// the tensor cores.  This kernel runs the same pipeline (TMA -> shared memory ring -> tcgen05.mma ->
// tensor memory -> selection warps, one thread per query row) with fp16 operands and fp16 accumulators:
// a selection thread pulls its 128 scores of a (key tile, query tile) pair out of tensor memory packed
// two to a register and reduces them with packed three-input maxima - half the registers and half the
// instructions per score.  What it computes is a FILTER, not the answer:
//   * Q and K are converted to fp16 after a power-of-two scaling per head that puts the largest row
//     norm into [32, 64) (f16_convert.cu), so nothing overflows and the conversion is exact except for
//     elements below 2^-14 of that;
//   * a candidate is a group of 8 keys - the even or the odd keys of a window of 16 consecutive keys,
//     which is what one packed register chain covers - ranked by the fp16 maximum of its scores;
//   * every row keeps the L best groups, L = k + slack (16, 24, 48 for k <= 8, 16, 32), in an unsorted
//     list in shared memory; a group that ties with the list's minimum is dropped;
//   * refine_f16.cu rescoring decides: it computes the exact fp32 scores of the kept groups' keys, proves
//     from the error bound of the fp16 scores that no dropped group can hold one of the k best keys, and
//     sends the rare row for which it cannot (more than L groups within the error bound of the k-th
//     best) to the exact CUDA-core kernel.
// The tensor cores round an fp16 accumulator to nearest after each 16-deep step (checked against the
// exact sums on the device), so |fp16 score - exact scaled score| <= 2^-11 (|partial sum| + |result|)
// for d = 32 and 2^-11 |result| for d = 16, plus the conversion's underflow terms.
//
// Warp roles, barriers, the ring of four 128-column accumulator buffers, the CTA-wide flush counter,
// the split tail of the persistent schedule and the bounded waits are those of score_select_tc.cu.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "f16_filter.cuh"
#include "ptx.cuh"

#include <cuda_fp16.h>

namespace kmip {

namespace {

constexpr int BM = 128;  // query rows per tile = TMEM lanes
constexpr int BN = 128;  // keys per tile = accumulator columns
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int NBUF = 4;  // accumulator buffers of BN columns: all 512 columns of tensor memory, used as a ring
constexpr int kRelaxedPollNs = 100;

template <int D>
struct Shape16 {
    static_assert(D == 16 || D == 32, "the fp16 prefilter covers head widths 16 and 32");
    static constexpr int RB = D * 2;                       // bytes per operand row = swizzle span
    static constexpr uint32_t LAYOUT = RB == 64 ? 4u : 6u;  // UMMA swizzle code (64-byte / 32-byte)
    static constexpr int KSTEPS = D / 16;                  // one tcgen05.mma covers 16 halves of depth
    static constexpr int TILE_BYTES = 128 * RB;
};

// Shared-memory matrix descriptor of a K-major, swizzled operand whose 8-row groups are contiguous.
template <int D>
__device__ __forceinline__ uint64_t make_desc16(uint32_t saddr) {
    using Sh = Shape16<D>;
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((8 * Sh::RB) >> 4) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of sm_100
    d |= (uint64_t)Sh::LAYOUT << 61;
    return d;
}

// Instruction descriptor: fp16 accumulate (format 0), fp16 A and B (format 0), both K-major, M = 128, N = BN.
constexpr uint32_t kInstrDesc16 = ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

template <int KG, int NQT, int S, int ROOM>
struct Plan16 {
    static constexpr int LIST = 8 * KG;  // groups kept per row
    // per row: LIST 16-bit scores, LIST 32-bit group words, ROOM pending 8-byte entries
    static constexpr int ROW_BYTES = 6 * LIST + 8 * ROOM;
    static constexpr int WARP_BYTES = 32 * ROW_BYTES;
    static constexpr int NBARS = 3 + 2 * S + NBUF * NQT + NBUF;
};

struct Bars {
    uint32_t base;
    int S, NQT;
    __device__ uint32_t q_full() const { return base; }
    __device__ uint32_t q_empty() const { return base + 8; }
    __device__ uint32_t done() const { return base + 16; }
    __device__ uint32_t k_full(int s) const { return base + 8 * (3 + s); }
    __device__ uint32_t k_empty(int s) const { return base + 8 * (3 + S + s); }
    __device__ uint32_t t_full(int b, int qt) const { return base + 8 * (3 + 2 * S + b * NQT + qt); }
    __device__ uint32_t t_empty(int b) const { return base + 8 * (3 + 2 * S + NBUF * NQT + b); }
};

template <int SLEEP_NS = 0>
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              StatusBlock* sb, int who, long long limit) {
    if (ptx::mbar_wait_bounded<SLEEP_NS>(bar, parity, abort_flag, limit)) return true;
    record_status(sb, KMIP_ERR_TIMEOUT, who);
    return false;
}

// fp16 bits <-> 16-bit unsigned integers that order like the numbers (0 = empty list slot).
__device__ __forceinline__ uint32_t order16(uint32_t h) { return (h ^ ((h & 0x8000u) ? 0xFFFFu : 0x8000u)) & 0xFFFFu; }
__device__ __forceinline__ uint32_t unorder16(uint32_t x) { return (x ^ ((x & 0x8000u) ? 0x8000u : 0xFFFFu)) & 0xFFFFu; }
constexpr uint32_t kHalfNegInf2 = 0xFC00FC00u, kHalfPosInf2 = 0x7C007C00u;

// Per-row selection state.  A warp's block of shared memory holds, slot-major so that lock-step loops
// are bank-conflict free: the score plane (slot s of lane l: 16 bits at s*64 + 2l), the group-word plane
// (32 bits at s*128 + 4l) and the pending entries (8 bytes at s*256 + 8l).  gmin caches the minimum of
// each 8-slot block of the list and lmin the minimum of the list, which stays 0 (empty) until LIST
// groups exist, so tau stays -inf until then.
template <int KG>
struct RowSel16 {
    uint32_t gmin[KG];
    uint32_t lmin;
    uint32_t tau2;  // the row's threshold in both halves: fp16 maximum of the LIST-th best group so far
    int cnt;
};

template <int KG>
__device__ __forceinline__ void row_init16(RowSel16<KG>& r, uint16_t* wl, int lane, bool rvalid) {
#pragma unroll 1
    for (int s = 0; s < 8 * KG; ++s) wl[s * 32 + lane] = 0;
#pragma unroll
    for (int g = 0; g < KG; ++g) r.gmin[g] = 0u;
    r.lmin = 0u;
    r.tau2 = rvalid ? kHalfNegInf2 : kHalfPosInf2;
    r.cnt = 0;
}

// All 32 lanes insert their pending groups into their own lists, in lock step.  A pending entry is
// {group word, packed register}: bit 31 of the word says which half of the register is the group's score.
template <int KG>
__device__ __forceinline__ void flush_pending16(RowSel16<KG>& r, uint32_t wl_s, uint32_t wk_s, uint32_t wp_s, bool rvalid) {
    const int maxc = __reduce_max_sync(FULL, r.cnt);
    __syncwarp();
#pragma unroll 1
    for (int t = 0; t < maxc; ++t) {
        if (t < r.cnt) {
            const uint2 raw = ptx::lds_v2(wp_s + (uint32_t)t * 256u);
            const uint32_t x = order16((raw.x >> 31) ? (raw.y >> 16) : (raw.y & 0xFFFFu));
            if (x > r.lmin) {
                int g = 0;
                uint32_t m = r.gmin[0];
#pragma unroll
                for (int q = 1; q < KG; ++q)
                    if (r.gmin[q] < m) { m = r.gmin[q]; g = q; }
                const uint32_t grp = wl_s + (uint32_t)g * (8u * 64u);
                uint32_t nm = x;
                int pos = -1;
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    const uint32_t y = ptx::lds_u16(grp + s * 64);
                    if (y == m && pos < 0) pos = s; else nm = min(nm, y);
                }
                ptx::sts_u16(grp + (uint32_t)pos * 64u, x);
                ptx::sts_u32(wk_s + (uint32_t)(g * 8 + pos) * 128u, raw.x);
#pragma unroll
                for (int q = 0; q < KG; ++q)
                    if (q == g) r.gmin[q] = nm;
                uint32_t lm = r.gmin[0];
#pragma unroll
                for (int q = 1; q < KG; ++q) lm = min(lm, r.gmin[q]);
                r.lmin = lm;
            }
        }
    }
    r.cnt = 0;
    if (rvalid) {
        const uint32_t t = r.lmin ? unorder16(r.lmin) : 0xFC00u;
        r.tau2 = t | (t << 16);
    }
}

// Packed maxima of a row's 128 scores: w[j] covers the 16-key window j (low half: its even keys, high
// half: its odd keys), q[c] the 32 keys of quad c, m the tile.  RAGGED: columns at or past `nvalid`
// do not exist (end of the key range).
template <bool RAGGED>
__device__ __forceinline__ void tile_maxima16(uint32_t (&v)[64], int nvalid, uint32_t (&w)[8], uint32_t (&q)[4], uint32_t& m) {
    if (RAGGED) {
#pragma unroll
        for (int x = 0; x < 64; ++x) {
            if (2 * x >= nvalid) v[x] = kHalfNegInf2;
            else if (2 * x + 1 >= nvalid) v[x] = (v[x] & 0xFFFFu) | 0xFC000000u;
        }
    }
    uint32_t a[8], b[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int o = 8 * j;
        a[j] = ptx::hmax3(v[o], v[o + 1], v[o + 2]);
        b[j] = ptx::hmax3(v[o + 3], v[o + 4], v[o + 5]);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = ptx::hmax3(v[8 * j + 6], v[8 * j + 7], a[j]);
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = ptx::hmax2(a[j], b[j]);
#pragma unroll
    for (int c = 0; c < 4; ++c) q[c] = ptx::hmax2(w[2 * c], w[2 * c + 1]);
    m = ptx::hmax2(ptx::hmax3(q[0], q[1], q[2]), q[3]);
}

// Lists the groups of a row's tile whose maximum beats tau.  Control flow is warp-uniform: a quad is
// visited when any lane has a hit in it (one vote); inside it each window costs one packed compare and
// two predicated (8-byte store, pointer bump) pairs.  `pend`: shared address of the lane's next free slot.
__device__ __forceinline__ void append_groups16(const uint32_t (&w)[8], const uint32_t (&q)[4], uint32_t tau2, int key0,
                                                uint32_t& pend) {
    unsigned hit[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) hit[c] = ptx::warp_ballot_half_gt(q[c], tau2);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (hit[c]) {
#pragma unroll
            for (int j = 2 * c; j < 2 * c + 2; ++j) {
                asm volatile(
                    "{\n\t"
                    ".reg .pred p, q;\n\t"
                    "setp.gt.f16x2 p|q, %1, %2;\n\t"
                    "@p st.shared.v2.b32 [%0], {%3, %1};\n\t"
                    "@p add.u32 %0, %0, 256;\n\t"
                    "@q st.shared.v2.b32 [%0], {%4, %1};\n\t"
                    "@q add.u32 %0, %0, 256;\n\t"
                    "}"
                    : "+r"(pend)
                    : "r"(w[j]), "r"(tau2), "r"(key0 + 16 * j), "r"((key0 + 16 * j) | 0x80000000u)
                    : "memory");
            }
        }
    }
}

template <int D, int KG, int NQT, int S, int ROOM, bool DUMP>
__global__ void __launch_bounds__(NQT * 128 + 96, 1)
score_select_f16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const WorkItem* __restrict__ items, StatusBlock* __restrict__ sb, int H,
                        uint32_t* __restrict__ cand_word, uint16_t* __restrict__ cand_half,
                        float* __restrict__ dump, int n_total /* = N */, long long wait_limit, int drop_first_tile,
                        const int* __restrict__ perm) {
    using Sh = Shape16<D>;
    using Sp = Plan16<KG, NQT, S, ROOM>;
    constexpr int NEPI = 4 * NQT;
    constexpr int NISS = 2;
    constexpr int LIST = Sp::LIST;
    constexpr uint32_t TMEM_COLS = NBUF * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + NQT * Sh::TILE_BYTES;
    uint8_t* sRows = sK + S * Sh::TILE_BYTES;
    uint64_t* sBars = reinterpret_cast<uint64_t*>(sRows + NEPI * Sp::WARP_BYTES);
    uint32_t* sTmem = reinterpret_cast<uint32_t*>(sBars + Sp::NBARS);
    volatile int* sAbort = reinterpret_cast<volatile int*>(sTmem + 1);
    volatile int* sFlushReq = reinterpret_cast<volatile int*>(sTmem + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Bars bars{ptx::smem_u32(sBars), S, NQT};

    if (threadIdx.x == 0) {
        ptx::mbar_init(bars.q_full(), 1);
        ptx::mbar_init(bars.q_empty(), NISS);
        ptx::mbar_init(bars.done(), NISS);
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(bars.k_full(s), 1);
            ptx::mbar_init(bars.k_empty(s), NQT);
        }
        for (int b = 0; b < NBUF; ++b) {
            for (int q = 0; q < NQT; ++q) ptx::mbar_init(bars.t_full(b, q), 1);
            ptx::mbar_init(bars.t_empty(b), 4);
        }
        *sAbort = 0;
        *sFlushReq = 0;
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
    // Tail of the persistent schedule: the units (work item, head) past the last full wave of CTAs are cut
    // into their 128-row query tiles, one CTA each, provided the pieces fit one wave (see score_select_tc.cu).
    long long n_whole = total, n_units = total;
    if (!DUMP && NQT > 1 && total > (long long)gridDim.x) {
        const long long left = total % gridDim.x;
        if (left * NQT <= (long long)gridDim.x) { n_whole = total - left; n_units = n_whole + left * NQT; }
    }
    auto unit = [&](long long w, int& h, WorkItem& it) -> bool {
        long long base = w;
        int piece = -1;
        if (w >= n_whole) { base = n_whole + (w - n_whole) / NQT; piece = (int)((w - n_whole) % NQT); }
        h = (int)(base / n_items);
        it = items[base % n_items];
        if (piece >= 0) { it.row0 += piece * BM; it.nrows = min(BM, it.nrows - piece * BM); }
        return it.nrows > 0;
    };

    if (warp == NEPI) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int kt = 0, ic = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < n_units; w += gridDim.x) {
                int h;
                WorkItem it;
                if (!unit(w, h, it)) continue;
                if (!(ok = wait_or_abort<kRelaxedPollNs>(bars.q_empty(), (ic & 1) ^ 1, sAbort, sb, 1, wait_limit))) break;
                ptx::mbar_arrive_expect_tx(bars.q_full(), NQT * Sh::TILE_BYTES);
                for (int qt = 0; qt < NQT; ++qt)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES), &tmQ, h * D, it.row0 + qt * BM, bars.q_full());
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; j < ntiles; ++j, ++kt) {
                    const int s = kt % S;
                    if (!(ok = wait_or_abort<kRelaxedPollNs>(bars.k_empty(s), ((kt / S) & 1) ^ 1, sAbort, sb, 2, wait_limit))) break;
                    // failure-detection test option: CTA 0 never loads its first key tile
                    if (drop_first_tile && blockIdx.x == 0 && kt == 0) continue;
                    ptx::mbar_arrive_expect_tx(bars.k_full(s), Sh::TILE_BYTES);
                    ptx::tma_load_2d(ptx::smem_u32(sK + s * Sh::TILE_BYTES), &tmK, 0, h * n_total + it.key_lo + j * BN,
                                     bars.k_full(s));
                }
                ++ic;
            }
            if (!ok) {
                // give copies that are still in flight a bounded time to land before the CTA exits
                const long long t0 = clock64();
                for (int s = 0; s < S && kt > 0; ++s) {
                    const int last = kt - 1 - ((kt - 1 - s) % S + S) % S;
                    if (last < 0) continue;
                    while (!ptx::mbar_try_wait(bars.k_full(s), (last / S) & 1) && clock64() - t0 < 40000000ll) {}
                }
            }
        }
    } else if (warp >= NEPI + 1 && warp <= NEPI + NISS) {
        // ------------------------------------------------------------------ MMA issuers
        // Pair number q of the CTA's (key tile, query tile) sequence uses accumulator buffer q mod 4; two
        // threads take the pairs alternately; the commit goes to a barrier per (buffer, query tile); both
        // issuers wait for every key tile (a parity wait is sound only on a barrier whose every phase the
        // waiter observes).
        if (lane == 0) {
            const int mine = warp - (NEPI + 1);
            uint64_t desc_q[NQT][Sh::KSTEPS], desc_k0[Sh::KSTEPS];
#pragma unroll
            for (int ks = 0; ks < Sh::KSTEPS; ++ks) {
#pragma unroll
                for (int qt = 0; qt < NQT; ++qt) desc_q[qt][ks] = make_desc16<D>(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + ks * 32));
                desc_k0[ks] = make_desc16<D>(ptx::smem_u32(sK + ks * 32));
            }
            int kt = 0, ic = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < n_units; w += gridDim.x) {
                int h_unused;
                WorkItem it;
                if (!unit(w, h_unused, it)) continue;
                const int nq = (it.nrows + BM - 1) / BM;
                if (!(ok = wait_or_abort<0>(bars.q_full(), ic & 1, sAbort, sb, 3, wait_limit))) break;
                ptx::tc_fence_after();
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; ok && j < ntiles; ++j, ++kt) {
                    const int s = kt % S;
                    const uint64_t stage_off = (uint64_t)((s * Sh::TILE_BYTES) >> 4);
                    if (!(ok = wait_or_abort<0>(bars.k_full(s), (kt / S) & 1, sAbort, sb, 4, wait_limit))) break;
#pragma unroll
                    for (int qt = 0; qt < NQT; ++qt) {
                        const int seq = kt * NQT + qt;
                        if ((seq & 1) != mine) continue;
                        const int b = seq & (NBUF - 1);
                        if (!(ok = wait_or_abort<0>(bars.t_empty(b), ((seq >> 2) & 1) ^ 1, sAbort, sb, 5, wait_limit))) break;
                        ptx::tc_fence_after();
                        if (qt < nq) {
                            const uint32_t d_tmem = tmem_base + (uint32_t)(b * BN);
#pragma unroll
                            for (int ks = 0; ks < Sh::KSTEPS; ++ks)
                                ptx::mma_f16_ss(d_tmem, desc_q[qt][ks], desc_k0[ks] + stage_off, kInstrDesc16, ks > 0 ? 1u : 0u);
                        }
                        ptx::mma_commit(bars.t_full(b, qt));
                    }
                }
                if (!ok) break;
                ptx::mma_commit(bars.q_empty());
                ++ic;
            }
            ptx::mma_commit(bars.done());
            const long long t0 = clock64();
            while (!ptx::mbar_try_wait(bars.done(), 0) && clock64() - t0 < 2000000000ll) {}
        }
    } else if (warp < NEPI) {
        // ------------------------------------------------------------------ selection warps
        const int qt = warp >> 2, quarter = warp & 3;
        uint8_t* wblock = sRows + (size_t)warp * Sp::WARP_BYTES;
        uint16_t* wl = reinterpret_cast<uint16_t*>(wblock);                    // score plane
        uint32_t* wk = reinterpret_cast<uint32_t*>(wblock + LIST * 64);        // group-word plane
        const uint32_t wl_s = ptx::smem_u32(wl + lane);
        const uint32_t wk_s = ptx::smem_u32(wk + lane);
        const uint32_t wp_addr = ptx::smem_u32(wblock + LIST * 192) + 8u * lane;  // this lane's first pending slot
        const uint32_t flush_req_s = ptx::smem_u32(const_cast<int*>(sFlushReq));
        const uint32_t full_bar0 = bars.t_full(0, qt);
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
        RowSel16<KG> rs;
        int flush_seen = 0;
        int tcnt = 0;
        bool ok = true;
        for (long long w = blockIdx.x; ok && w < n_units; w += gridDim.x) {
            int h;
            WorkItem it;
            if (!unit(w, h, it)) continue;
            const bool active = qt * BM < it.nrows;
            const int local = qt * BM + quarter * 32 + lane;
            const bool rvalid = local < it.nrows;
            if (active) row_init16<KG>(rs, wl, lane, rvalid);
            __syncwarp();
            const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
            constexpr int kUseShift = NQT == 2 ? 1 : 2;
            if (DUMP || !active) {
                for (int j = 0; j < ntiles; ++j, ++tcnt) {
                    const int b = (tcnt * NQT + qt) & (NBUF - 1);
                    ok = wait_or_abort(full_bar0 + (uint32_t)b * (8u * NQT), (uint32_t)(tcnt >> kUseShift) & 1u, sAbort, sb,
                                       6, wait_limit);
                    ok = __all_sync(FULL, ok);
                    if (!ok) break;
                    if (quarter == 0 && lane == 0) ptx::mbar_arrive(bars.k_empty(tcnt % S));
                    ptx::tc_fence_after();
                    if (DUMP && active) {
                        const int key0 = it.key_lo + j * BN;
                        const int ncol = min(BN, it.key_hi - key0);
                        uint32_t v[64];
                        ptx::tmem_ld_32x128_pack16_sync(taddr0 + (uint32_t)(b * BN), v);
                        if (rvalid) {
#pragma unroll
                            for (int x = 0; x < 64; ++x) {
                                float* o = dump + ((size_t)h * n_total + it.row0 + local) * n_total + key0 + 2 * x;
                                if (2 * x < ncol) o[0] = __half2float(__ushort_as_half((unsigned short)(v[x] & 0xFFFFu)));
                                if (2 * x + 1 < ncol) o[1] = __half2float(__ushort_as_half((unsigned short)(v[x] >> 16)));
                            }
                        }
                    }
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));
                }
            } else {
                const int ragged_j = ((it.key_hi - it.key_lo) & (BN - 1)) ? ntiles - 1 : -1;
                int key0 = it.key_lo;
                for (int j = 0; j < ntiles; ++j, ++tcnt, key0 += BN) {
                    const int b = (tcnt * NQT + qt) & (NBUF - 1);
                    const uint32_t full_bar = full_bar0 + (uint32_t)b * (8u * NQT);
                    const uint32_t full_par = (uint32_t)(tcnt >> kUseShift) & 1u;
                    if (!__all_sync(FULL, ptx::mbar_try_wait(full_bar, full_par))) {
                        // scores not there yet: merge pending groups meanwhile, then block
                        if (__any_sync(FULL, rs.cnt > 0)) flush_pending16<KG>(rs, wl_s, wk_s, wp_addr, rvalid);
                        ok = wait_or_abort(full_bar, full_par, sAbort, sb, 6, wait_limit);
                        ok = __all_sync(FULL, ok);
                        if (!ok) break;
                    }
                    if (quarter == 0 && lane == 0) ptx::mbar_arrive(bars.k_empty(tcnt % S));
                    ptx::tc_fence_after();
                    uint32_t v[64], wm[8], qm[4], m;
                    ptx::tmem_ld_32x128_pack16_sync(taddr0 + (uint32_t)(b * BN), v);
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));  // the buffer goes straight back to the issuers
                    if (j == ragged_j) tile_maxima16<true>(v, it.key_hi - key0, wm, qm, m);
                    else tile_maxima16<false>(v, BN, wm, qm, m);
                    const int req = (int)ptx::lds_u32(flush_req_s);
                    bool do_flush = req != flush_seen;
                    if (ptx::warp_any_half_gt(m, rs.tau2)) {  // some lane of the warp has a hit in this tile
                        uint32_t pend = wp_addr + (uint32_t)rs.cnt * 256u;
                        append_groups16(wm, qm, rs.tau2, key0, pend);
                        rs.cnt = (int)((pend - wp_addr) >> 8);
                        if (__any_sync(FULL, rs.cnt > ROOM - 16)) {  // a tile adds at most 16 groups per row
                            do_flush = true;
                            if (lane == 0 && req == flush_seen) atomicAdd(const_cast<int*>(sFlushReq), 1);
                        }
                    }
                    if (do_flush) {
                        flush_pending16<KG>(rs, wl_s, wk_s, wp_addr, rvalid);
                        flush_seen = req + ((req == flush_seen) ? 1 : 0);
                    }
                }
            }
            if (!ok) break;
            if (!DUMP && active) {
                // finalise: drain the pending slots, then store each row's LIST groups (group word and fp16
                // maximum, unsorted; empty slots as all-ones / -inf) for the rescoring kernel
                flush_pending16<KG>(rs, wl_s, wk_s, wp_addr, rvalid);
                __syncwarp();
                const int nloc = min(32, it.nrows - (qt * BM + quarter * 32));
                for (int r = 0; r < nloc; ++r) {
                    const int srow = it.row0 + qt * BM + quarter * 32 + r;  // sweep order; the result goes to the row's own place
                    const int orow = perm ? __ldg(perm + srow) : srow;
                    if (!kmip_check(orow >= 0 && orow < n_total, sb, 103)) continue;  // checks builds: a row of the batch
                    const size_t o = ((size_t)orow * H + h) * LIST;
                    for (int t = lane; t < LIST; t += 32) {
                        const uint32_t c = wl[t * 32 + r];
                        cand_word[o + t] = c ? wk[t * 32 + r] : 0xFFFFFFFFu;
                        cand_half[o + t] = (uint16_t)(c ? unorder16(c) : 0xFC00u);
                    }
                }
                __syncwarp();
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

// Tensor map over an fp16 matrix of `rows` rows of `row_elems` elements; a box is 128 rows x D columns.
template <int D>
bool make_tensor_map16(CUtensorMap* tm, const void* base, int64_t rows, int64_t row_elems) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)row_elems, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)row_elems * 2};
    const cuuint32_t box[2] = {(cuuint32_t)D, 128u};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUtensorMapSwizzle sw = D == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int KG, int NQT, int S, int ROOM, bool DUMP>
cudaError_t launch_cfg(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    using Sh = Shape16<D>;
    using Sp = Plan16<KG, NQT, S, ROOM>;
    constexpr size_t smem_bytes = 1024 + (size_t)(NQT + S) * Sh::TILE_BYTES + (size_t)4 * NQT * Sp::WARP_BYTES +
                                  (size_t)Sp::NBARS * 8 + 64;
    static_assert(smem_bytes <= 232448, "shared memory budget of one CTA");
    CUtensorMap tmQ, tmK;
    if (!make_tensor_map16<D>(&tmQ, a.ws + w.qperm_off, a.N, (int64_t)a.H * D) ||
        !make_tensor_map16<D>(&tmK, a.ws + w.kpack_off, a.N * a.H, D))
        return cudaErrorInvalidValue;
    auto kern = score_select_f16_kernel<D, KG, NQT, S, ROOM, DUMP>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (err != cudaSuccess) return err;
    const long long max_total = (long long)w.max_items * a.H;
    const int grid = (int)std::min<long long>(sm_count(), max_total);
    kern<<<grid, NQT * 128 + 96, smem_bytes, a.stream>>>(
        tmQ, tmK, reinterpret_cast<const WorkItem*>(a.ws + w.items_off), reinterpret_cast<StatusBlock*>(a.ws), a.H,
        reinterpret_cast<uint32_t*>(a.ws + w.cand_word_off), reinterpret_cast<uint16_t*>(a.ws + w.cand_half_off), dump,
        (int)a.N, a.wait_limit_cycles > 0 ? a.wait_limit_cycles : kDefaultWaitLimitCycles, a.drop_first_tile,
        (w.reorder && !DUMP) ? reinterpret_cast<const int*>(a.ws + w.perm_off) : nullptr);
    return cudaGetLastError();
}

template <int D, bool DUMP>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    // (list blocks, query tiles per CTA, key stages, pending slots per row); shared memory decides
    // the per-warp block of shared memory stays at 14848 bytes: 192 per list slot, 256 per pending slot
    return launch_cfg<D, kF16List32 / 8, 3, 3, (14848 - kF16List32 * 192) / 256, DUMP>(a, w, dump);
}

}  // namespace

bool score_select_f16_supported(int32_t d, int32_t k) { return (d == 16 || d == 32) && k <= 32; }
int score_select_f16_list(int32_t k) { return k <= 8 ? 16 : k <= 16 ? 24 : kF16List32; }
// lists of up to 24 groups (k <= 16) run the four-pipeline kernel of score_select_f16x4.cu with 512-row work items
int score_select_f16_rows_per_item(int32_t k) { return k <= 16 ? score_select_f16x4_rows_per_item() : 3 * BM; }

cudaError_t launch_score_select_f16(const FwdArgs& a, const FwdWorkspace& w) {
    if (a.k <= 16) return launch_score_select_f16x4(a, w);
    return a.d == 16 ? launch_d<16, false>(a, w, nullptr) : launch_d<32, false>(a, w, nullptr);
}

}  // namespace kmip
