// Tensor-core score + running top-k kernel (Algorithm 1 lines 2-3) for sm_100a.
//
// The paper evaluates S = Q K^T lazily (a "symbolic matrix") on CUDA cores and reduces each row
// to its k best entries without storing S.  Here the same reduction is fed by the 5th-generation
// tensor cores: a persistent CTA per SM owns up to 384 query rows (NQT 128-row tiles) of one
// graph and one head, streams that graph's keys in 128-key tiles through a TMA -> shared memory
// ring, multiplies each key tile against every query tile with tcgen05.mma (bf16 in, fp32
// accumulators in tensor memory: four 128-column buffers used as a ring by the sequence of
// (key tile, query tile) pairs), and 4*NQT selection warps read the accumulators straight out of
// tensor memory.  One thread owns one query row.
//   fast pass   the thread pulls its 128 scores of the pair into registers (the accumulator
//               buffer goes straight back to the MMA issuers), reduces every 8 consecutive
//               columns to their maximum with three-input max instructions and compares the
//               tile maximum once against the row's threshold tau;
//   candidates  a candidate is an 8-key GROUP, ranked by its maximum.  The k groups with the
//               largest maxima always contain k keys whose scores are the k largest of the row:
//               if a key of the top k sat in a group outside them, each of the k groups would
//               hold a key at least as good.  So the sweep only tracks groups: a lane whose tile
//               maximum beats tau appends (group maximum, first key) for the groups above tau to
//               its pending slots - no index search.  Groups with EQUAL maxima are not ordered
//               further (a new one never displaces an equal old one); the rescoring kernel applies
//               the (score desc, key asc) order to the keys it is given;
//   flush       when a pending area fills up all 32 lanes insert their pending groups into their
//               own unsorted k-entry lists in lock step (replace the list minimum, 8-slot blocks
//               with cached minima) and refresh tau = k-th best group maximum so far.
// When an item ends each row's k groups go to global memory; refine.cu rescores their 8k keys
// exactly and keeps the best k.  The N x N scores never leave the SM.
//
// Warp roles (NQT = query tiles per CTA, 1 to 3):
//   warps 0 .. 4*NQT-1   selection; warp w reads TMEM lanes 32*(w%4).. for query tile w/4
//   warp 4*NQT           TMA producer (one lane)
//   warps 4*NQT+1, +2    tcgen05.mma issue (one lane each, alternating pairs); +1 owns TMEM
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

constexpr int kRelaxedPollNs = 100;  // sleep between polls of the waits that are off the critical path
constexpr int NBUF = 4;  // accumulator buffers of BN columns: all 512 columns of tensor memory, used as a ring

template <int KG, int NQT, int S>
struct SmemPlan {
    static constexpr int LIST = 8 * KG;               // list slots per row (k <= LIST)
    static constexpr int ROOM = (NQT >= 3 || (NQT == 2 && KG >= 8)) ? 24 : 32;  // pending candidate slots per row (a tile adds at most 16)
    static constexpr int SLOTS = LIST + ROOM;         // cand_t per row
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

// SLEEP_NS > 0: the waiter is off the critical path (the TMA producer and the MMA issuers run
// well ahead of the selection warps) and sleeps between polls instead of competing for issue slots.
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              StatusBlock* sb, int who, long long limit) {
    if (ptx::mbar_wait_bounded<SLEEP_NS>(bar, parity, abort_flag, limit)) return true;
    record_status(sb, KMIP_ERR_TIMEOUT, who);
    return false;
}

// Per-row selection state of one thread.  The row's slots live in the warp's block of shared
// memory in slot-major order (slot s of lane l at [s*32 + l]), so lock-step loops over slots are
// bank-conflict free.  The k-entry list is unsorted and split into two 32-bit planes: the order-
// preserving bits of the group maximum (0 = empty slot, ~0 = slot past k) and the group's first
// key.  gmin caches the minimum of each 8-slot block and lmin the minimum of the list, so tau stays
// -inf until k real entries exist.  Only the score plane takes part in comparisons: a candidate
// must beat the list minimum strictly, so of two groups with equal maxima the one met first (the
// lower keys) stays; among several list entries that tie for the minimum the first slot is replaced.
template <int KG>
struct RowSel {
    uint32_t gmin[KG];
    uint32_t lmin;
    float tau;
    int cnt;
};

template <int KG>
__device__ __forceinline__ void row_init(RowSel<KG>& r, uint32_t* wl, int k, int lane, bool rvalid) {
#pragma unroll 1
    for (int s = 0; s < 8 * KG; ++s) wl[s * 32 + lane] = (s < k) ? 0u : ~0u;  // slots past k are never the minimum
#pragma unroll
    for (int g = 0; g < KG; ++g) r.gmin[g] = (8 * g < k) ? 0u : ~0u;
    r.lmin = 0u;
    r.tau = rvalid ? -CUDART_INF_F : CUDART_INF_F;
    r.cnt = 0;
}

// All 32 lanes insert their pending candidates into their own lists, in lock step.  `wl_s` is the
// shared address of the lane's slot 0 in the score plane of the warp's lists (slots 128 bytes
// apart, the key plane 8*KG*128 bytes further), `wp_s` that of the lane's first pending slot
// (256 bytes apart).
template <int KG>
__device__ __forceinline__ void flush_pending(RowSel<KG>& r, uint32_t wl_s, uint32_t wp_s, bool rvalid) {
    const int maxc = __reduce_max_sync(FULL, r.cnt);
    __syncwarp();
#pragma unroll 1
    for (int t = 0; t < maxc; ++t) {
        if (t < r.cnt) {
            const uint2 raw = ptx::lds_v2(wp_s + (uint32_t)t * 256u);  // {first key, fp32 bits}
            const uint32_t x = order_bits(__uint_as_float(raw.y) + 0.0f);
            if (x > r.lmin) {
                int g = 0;
                uint32_t m = r.gmin[0];
#pragma unroll
                for (int q = 1; q < KG; ++q)
                    if (r.gmin[q] < m) { m = r.gmin[q]; g = q; }
                const uint32_t grp = wl_s + (uint32_t)g * (8u * 128u);
                uint32_t nm = x;
                int pos = -1;
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    const uint32_t y = ptx::lds_u32(grp + s * 128);
                    if (y == m && pos < 0) pos = s; else nm = min(nm, y);
                }
                ptx::sts_u32(grp + (uint32_t)pos * 128u, x);
                ptx::sts_u32(grp + (uint32_t)pos * 128u + 8u * KG * 128u, raw.x);
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
    if (rvalid) r.tau = r.lmin ? unorder_bits(r.lmin) : -CUDART_INF_F;
}

// Maxima of the eight 8-column groups of 64 consecutive columns (three-input max; all first-level
// operations come before the second level so that they issue back to back), and of the two
// 32-column quads.  RAGGED: columns at or past `nvalid` do not exist (end of the key range).
template <bool RAGGED>
__device__ __forceinline__ void half_maxima(uint32_t (&v)[64], int nvalid, float* sub, float* quad) {
    if (RAGGED) {
#pragma unroll
        for (int x = 0; x < 64; ++x)
            if (x >= nvalid) v[x] = 0xFF800000u;  // -inf
    }
    float m0[8], m1[8], m2[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const int o = 8 * g;
        m0[g] = ptx::max3(__uint_as_float(v[o]), __uint_as_float(v[o + 1]), __uint_as_float(v[o + 2]));
        m1[g] = ptx::max3(__uint_as_float(v[o + 3]), __uint_as_float(v[o + 4]), __uint_as_float(v[o + 5]));
        m2[g] = fmaxf(__uint_as_float(v[o + 6]), __uint_as_float(v[o + 7]));
    }
#pragma unroll
    for (int g = 0; g < 8; ++g) sub[g] = ptx::max3(m0[g], m1[g], m2[g]);
    quad[0] = fmaxf(ptx::max3(sub[0], sub[1], sub[2]), sub[3]);
    quad[1] = fmaxf(ptx::max3(sub[4], sub[5], sub[6]), sub[7]);
}

// Lists the groups of a row's tile that beat tau.  Control flow is warp-uniform: a 32-column quad is
// visited when any lane has a hit in it (one vote), and inside a quad each group costs one compare,
// one predicated 8-byte store and one predicated pointer bump.  A pending entry is {first key of
// the group, raw fp32 bits of the group maximum}; `pend` is the shared-memory byte address of the
// lane's next free slot (256 bytes apart).
__device__ __forceinline__ void append_groups(const float (&sub)[16], const float (&quad)[4], float tau, int key_base,
                                              uint32_t& pend) {
    // four independent votes first, warp-uniform branches afterwards
    unsigned hit[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) hit[c] = __ballot_sync(FULL, quad[c] > tau);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (hit[c]) {
#pragma unroll
            for (int g = 4 * c; g < 4 * c + 4; ++g) {
                asm volatile(
                    "{\n\t"
                    ".reg .pred p;\n\t"
                    "setp.gt.f32 p, %1, %2;\n\t"
                    "@p st.shared.v2.b32 [%0], {%3, %1};\n\t"
                    "@p add.u32 %0, %0, 256;\n\t"
                    "}"
                    : "+r"(pend)
                    : "f"(sub[g]), "f"(tau), "r"(key_base + 8 * g)
                    : "memory");
            }
        }
    }
}

// What the pruned sweep (PRUNE) adds to the kernel below.  The TMA producer decides, 32 key tiles at a
// time (one per lane), which tiles no row of the CTA's query block can take a candidate from (bounds of
// prune.cu against the thresholds the selection warps publish per warp) and loads only the others, so the
// tiles that flow through the pipeline are no longer numbered consecutively:
//   * the producer writes each loaded tile's first key into sStageKey[stage] before it arms the stage's
//     full barrier, and ends an item with a pseudo tile (first key -1, no data, a plain arrive);
//   * an issuer reads it after the full-barrier wait, acknowledges the read with an arrival of its own on
//     the stage's empty barrier (with one query tile per CTA an issuer owns no pair of every other tile
//     and would otherwise read the stage after it was refilled), copies it to sBufKey[buffer] before the
//     pair's commit (or, for the pseudo tile, a plain arrive on the pair's barrier) and leaves the item
//     after the pseudo tile;
//   * a selection warp reads sBufKey[buffer] after its wait and before it hands the buffer back.
// A skipped tile would have produced no candidate: every group maximum in it is below the row's
// threshold at decision time, and thresholds only rise.  So the lists are those of the full sweep.
struct PruneArgs {
    const float* qstat;  // [items, H, D+4]
    const float* kstat;  // [tiles, H, D+4]
    const float* qnorm;  // [N, H], sweep order
};

constexpr int kPruneTilesPerLane = 1;  // key tiles a producer lane decides per batch (4: staler thresholds, 4 % slower)
constexpr int kEndOfItem = -1;  // "first key" of the pseudo tile that ends an item
constexpr int kDeadPair = -2;   // "first key" of a (key tile, query tile) pair the bounds ruled out

// A selection warp tells the producer the smallest threshold of its rows and the smallest
// threshold / |q| (only rows with a positive threshold can use the norm bound), tagged with the item.
__device__ __forceinline__ void publish_thresholds(float tau, float inv_qn, int ic, uint32_t stat_s, int lane) {
    const float ratio = tau > 0.0f ? tau * inv_qn : -CUDART_INF_F;  // rows past the item's end have tau = +inf
    const uint32_t tm = __reduce_min_sync(FULL, order_bits(tau));
    const uint32_t rm = __reduce_min_sync(FULL, order_bits(ratio));
    if (lane == 0) {
        ptx::sts_v2(stat_s, (uint32_t)ic, __float_as_uint(unorder_bits(tm)));
        ptx::sts_v2(stat_s + 8u, (uint32_t)ic, __float_as_uint(unorder_bits(rm)));
    }
}

// LSE: instead of selecting, the selection warps fold every score of a row into a running log-sum-exp
// (base 2, scale log2(e)/sqrt(d)) and write the share of the full softmax that the row's k kept scores
// hold - the cumulative-attention-weight diagnostic of the paper's appendix "Additional results" - to
// `dump` as float [N, H]; `topk_score` is then an input.
template <int D, int KG, int NQT, int S, bool DUMP, bool PRUNE, bool LSE = false>
__global__ void __launch_bounds__(NQT * 128 + 96, 1)
score_select_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const WorkItem* __restrict__ items, StatusBlock* __restrict__ sb, int H, int k,
                       int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                       float* __restrict__ dump, int dump_ld /* = N */, long long wait_limit, int drop_first_tile,
                       const int* __restrict__ perm, const PruneArgs pr) {
    static_assert(!(DUMP && PRUNE) && !(LSE && (DUMP || PRUNE)), "the score dump and the softmax-share pass sweep every tile");
    using Sh = TcShape<D>;
    using Sp = SmemPlan<KG, NQT, S>;
    constexpr int NEPI = 4 * NQT;
    constexpr int NISS = 2;  // MMA issuer threads (see the issuer branch)
    constexpr int ROOM = Sp::ROOM;
    constexpr uint32_t TMEM_COLS = NBUF * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + NQT * Sh::TILE_BYTES;
    cand_t* sRows = reinterpret_cast<cand_t*>(sK + S * Sh::TILE_BYTES);
    uint64_t* sBars = reinterpret_cast<uint64_t*>(sRows + NQT * 128 * Sp::SLOTS);
    uint32_t* sTmem = reinterpret_cast<uint32_t*>(sBars + Sp::NBARS);
    volatile int* sAbort = reinterpret_cast<volatile int*>(sTmem + 1);
    volatile int* sFlushReq = reinterpret_cast<volatile int*>(sTmem + 2);  // CTA-wide flush request counter
    volatile int* sStageKey = reinterpret_cast<volatile int*>(sTmem + 4);   // [4] first key of the tile in a key stage
    volatile int* sBufKey = reinterpret_cast<volatile int*>(sTmem + 8);     // [4] first key of the pair in an accumulator buffer
    // [warp][2] {item number, float bits}: smallest threshold and smallest threshold / query norm of the warp's rows
    const uint32_t warp_stat_s = ptx::smem_u32(sTmem + 12);
    volatile int* sStageDead = reinterpret_cast<volatile int*>(sTmem + 60);  // [4] query tiles that skip the stage's key tile (bit mask)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Bars bars{ptx::smem_u32(sBars), S, NQT};

    if (threadIdx.x == 0) {
        ptx::mbar_init(bars.q_full(), 1);
        ptx::mbar_init(bars.q_empty(), NISS);  // every MMA issuer commits to it
        ptx::mbar_init(bars.done(), NISS);
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(bars.k_full(s), 1);
            ptx::mbar_init(bars.k_empty(s), NQT + (PRUNE ? NISS : 0));  // one arrival per query tile (and per issuer's read)
        }
        for (int b = 0; b < NBUF; ++b) {
            for (int q = 0; q < NQT; ++q) ptx::mbar_init(bars.t_full(b, q), 1);
            ptx::mbar_init(bars.t_empty(b), 4);  // the four selection warps of the query tile that read the buffer
        }
        *sAbort = 0;
        *sFlushReq = 0;
        if (PRUNE)
            for (int i = 0; i < 2 * NEPI; ++i) ptx::sts_v2(warp_stat_s + 8u * i, 0xFFFFFFFFu, 0u);  // item number -1: not valid
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
    // Tail of the persistent schedule.  A unit of work is a (work item, head) pair and takes the same time
    // whether one or all of its query tiles hold rows (the warp groups run side by side), so when the units
    // do not divide by the grid, the last `left` ones would keep a few CTAs busy for a whole unit while the
    // rest idle.  Those units are cut into their 128-row query tiles instead, one CTA each - a CTA with a
    // single busy warp group gets through its key tiles faster - provided the pieces fit one wave.
    long long n_whole = total, n_units = total;
    if (!PRUNE && !DUMP && !LSE && NQT > 1 && total > (long long)gridDim.x) {
        const long long left = total % gridDim.x;
        if (left * NQT <= (long long)gridDim.x) { n_whole = total - left; n_units = n_whole + left * NQT; }
    }
    // unit number -> head and work item (all roles decode it the same way); false: a piece without rows
    auto unit = [&](long long w, int& h, WorkItem& it) -> bool {
        long long base = w;
        int piece = -1;
        if (w >= n_whole) { base = n_whole + (w - n_whole) / NQT; piece = (int)((w - n_whole) % NQT); }
        h = (int)(base / n_items);
        it = items[base % n_items];
        if (piece >= 0) { it.row0 += piece * BM; it.nrows = min(BM, it.nrows - piece * BM); }
        return it.nrows > 0;
    };

    if (PRUNE && warp == NEPI) {
        // ------------------------------------------------------------------ TMA producer, pruned sweep
        // All 32 lanes evaluate bounds (one tile each); lane 0 runs the pipeline.
        constexpr int REC = D + 4;
        int kt = 0, ic = 0;
        bool ok = true;
        long long n_all = 0, n_pairs_all = 0, n_pairs_live = 0;  // counters for the optional statistics buffer
        for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
            const int h = (int)(w / n_items);
            const int item = (int)(w % n_items);
            const WorkItem it = items[item];
            if (lane == 0) {
                ok = wait_or_abort<kRelaxedPollNs>(bars.q_empty(), (ic & 1) ^ 1, sAbort, sb, 1, wait_limit);
                if (ok) {
                    ptx::mbar_arrive_expect_tx(bars.q_full(), NQT * Sh::TILE_BYTES);
                    for (int qt = 0; qt < NQT; ++qt)
                        for (int ch = 0; ch < Sh::KCH; ++ch)
                            ptx::tma_load_2d(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmQ,
                                             h * D + ch * 64, it.row0 + qt * BM, bars.q_full());
                }
            }
            ok = __shfl_sync(FULL, (int)ok, 0) != 0;
            if (!ok) break;
            // one record per 128-row query tile of the item: centroid, radius, centroid norm (all lanes read
            // the same addresses); the first record also holds the tile the sweep starts at
            const float* qrec0 = pr.qstat + ((size_t)item * NQT * H + h) * REC;
            const int nq = (it.nrows + BM - 1) / BM;  // query tiles that hold rows
            const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
            // The sweep starts at the tile the statistics kernel chose for the block, runs to the end of the
            // graph and then takes the tiles in front of the start.
            const int jstart = min(max(__float_as_int(__ldg(qrec0 + D + 3)), 0), ntiles - 1);
            n_all += ntiles;
            n_pairs_all += (long long)ntiles * nq;
            // query tiles (bit mask) that cannot take a candidate from key tile j; `rest` is set when that holds
            // for tile j and every later tile of the graph by the norm bound alone
            auto evaluate = [&](int j, bool& rest) -> unsigned {
                unsigned dead = (1u << NQT) - 1u;
                const float4* krec = reinterpret_cast<const float4*>(pr.kstat + ((size_t)(it.tile0 + j) * H + h) * REC);
                float4 ck[D / 4];
#pragma unroll
                for (int c = 0; c < D / 4; ++c) ck[c] = __ldg(krec + c);
                const float4 ktail = __ldg(krec + D / 4);
                const float r_t = ktail.x, n_ct = ktail.y, k_max = ktail.z, k_max_rest = ktail.w;
                rest = true;
#pragma unroll
                for (int qt = 0; qt < NQT; ++qt) {
                    if (qt >= nq) continue;  // no rows: nothing to object
                    const float4* qrec = reinterpret_cast<const float4*>(qrec0 + (size_t)qt * H * REC);
                    float dot = 0.0f;
#pragma unroll
                    for (int c = 0; c < D / 4; ++c) {
                        const float4 t = __ldg(qrec + c);
                        dot = fmaf(ck[c].x, t.x, dot); dot = fmaf(ck[c].y, t.y, dot);
                        dot = fmaf(ck[c].z, t.z, dot); dot = fmaf(ck[c].w, t.w, dot);
                    }
                    const float4 qtail = __ldg(qrec + D / 4);
                    const float r_b = qtail.x, n_cq = qtail.y;
                    const float spread = n_cq * r_t + n_ct * r_b + r_b * r_t;
                    // rounding of the bound itself and of the tensor-core scores, both relative to |q| |k|
                    const float bound = dot + spread + 1e-4f * (n_cq * n_ct + spread);
                    // thresholds published for THIS item; a warp that has not started it yet counts as -inf
                    float tau_min = CUDART_INF_F, ratio_min = CUDART_INF_F;
#pragma unroll
                    for (int wq = 4 * qt; wq < 4 * qt + 4; ++wq) {
                        const uint2 a = ptx::lds_v2(warp_stat_s + 16u * wq);
                        const uint2 b = ptx::lds_v2(warp_stat_s + 16u * wq + 8u);
                        tau_min = fminf(tau_min, (int)a.x == ic ? __uint_as_float(a.y) : -CUDART_INF_F);
                        ratio_min = fminf(ratio_min, (int)b.x == ic ? __uint_as_float(b.y) : -CUDART_INF_F);
                    }
                    if (!(bound < tau_min || k_max < ratio_min)) dead &= ~(1u << qt);
                    rest = rest && k_max_rest < ratio_min;
                }
                return dead;
            };
            // Decisions are taken for a batch of tiles at a time (lane l: tiles l, l + 32, ...) and the batch
            // is then fed to the pipeline by lane 0; the first batch of an item is small because nothing can
            // be skipped before the first thresholds exist.
            constexpr int U = kPruneTilesPerLane;
            bool first_batch = true;
            for (int seg = 0; ok && seg < 2; ++seg) {
                const int seg_hi = seg == 0 ? ntiles : jstart;
                for (int j0 = seg == 0 ? jstart : 0; ok && j0 < seg_hi;) {
                    const int nbatch = min(first_batch ? 32 : 32 * U, seg_hi - j0);
                    first_batch = false;
                    unsigned dead[U];
                    bool seg_done = false;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        dead[u] = (1u << NQT) - 1u;
                        bool rest = false;
                        if (u * 32 + lane < nbatch) dead[u] = evaluate(j0 + u * 32 + lane, rest);
                        seg_done = seg_done || __any_sync(FULL, rest);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (u * 32 >= nbatch) break;
                        const unsigned skip_mask = __ballot_sync(FULL, dead[u] == (1u << NQT) - 1u);
                        const int nb = min(32, nbatch - u * 32);
                        for (int l = 0; l < nb; ++l) {
                            const unsigned dead_l = __shfl_sync(FULL, dead[u], l);
                            if (lane != 0 || ((skip_mask >> l) & 1u) || !ok) continue;
                            const int s = kt % S;
                            if (!(ok = wait_or_abort<kRelaxedPollNs>(bars.k_empty(s), ((kt / S) & 1) ^ 1, sAbort, sb, 2, wait_limit))) continue;
                            const int key0 = it.key_lo + (j0 + u * 32 + l) * BN;
                            sStageKey[s] = key0;
                            sStageDead[s] = (int)dead_l;
                            n_pairs_live += nq - __popc(dead_l & ((1u << nq) - 1u));
                            ptx::mbar_arrive_expect_tx(bars.k_full(s), Sh::TILE_BYTES);
                            for (int ch = 0; ch < Sh::KCH; ++ch)
                                ptx::tma_load_2d(ptx::smem_u32(sK + s * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmK,
                                                 ch * 64, h * dump_ld + key0, bars.k_full(s));
                            ++kt;
                        }
                    }
                    ok = __shfl_sync(FULL, (int)ok, 0) != 0;
                    kt = __shfl_sync(FULL, kt, 0);
                    if (seg_done) break;  // every tile after the first dead one was skipped by the same test
                    j0 += nbatch;
                }
            }
            if (!ok) break;
            if (lane == 0) {
                // the pseudo tile that ends the item: no data, the phase completes with this arrive
                const int s = kt % S;
                ok = wait_or_abort<kRelaxedPollNs>(bars.k_empty(s), ((kt / S) & 1) ^ 1, sAbort, sb, 2, wait_limit);
                if (ok) {
                    sStageKey[s] = kEndOfItem;
                    ptx::mbar_arrive(bars.k_full(s));
                    ++kt;
                }
            }
            ok = __shfl_sync(FULL, (int)ok, 0) != 0;
            kt = __shfl_sync(FULL, kt, 0);
            ++ic;
        }
        if (lane == 0) {  // key tiles of the CTA's items, tiles loaded (with the end markers), pairs, pairs scored
            atomicAdd(&sb->counters[0], (unsigned long long)n_all);
            atomicAdd(&sb->counters[1], (unsigned long long)kt);
            atomicAdd(&sb->counters[2], (unsigned long long)n_pairs_all);
            atomicAdd(&sb->counters[3], (unsigned long long)n_pairs_live);
        }
        if (!ok && lane == 0) {
            // give copies that are still in flight a bounded time to land before the CTA exits; a stage
            // whose last use was a pseudo tile has completed that phase already
            const long long t0 = clock64();
            for (int s = 0; s < S && kt > 0; ++s) {
                const int last = kt - 1 - ((kt - 1 - s) % S + S) % S;
                if (last < 0) continue;
                while (!ptx::mbar_try_wait(bars.k_full(s), (last / S) & 1) && clock64() - t0 < 40000000ll) {}
            }
        }
    } else if (warp == NEPI) {
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
                    for (int ch = 0; ch < Sh::KCH; ++ch)
                        ptx::tma_load_2d(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmQ,
                                         h * D + ch * 64, it.row0 + qt * BM, bars.q_full());
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; j < ntiles; ++j, ++kt) {
                    const int s = kt % S;
                    if (!(ok = wait_or_abort<kRelaxedPollNs>(bars.k_empty(s), ((kt / S) & 1) ^ 1, sAbort, sb, 2, wait_limit))) break;
                    // failure-detection test hook: CTA 0 never loads its first key tile, so the waits on
                    // that stage must run out, be reported and leave the context usable
                    if (drop_first_tile && blockIdx.x == 0 && kt == 0) continue;
                    ptx::mbar_arrive_expect_tx(bars.k_full(s), Sh::TILE_BYTES);
                    for (int ch = 0; ch < Sh::KCH; ++ch)
                        ptx::tma_load_2d(ptx::smem_u32(sK + s * Sh::TILE_BYTES + ch * Sh::CH_BYTES), &tmK,
                                         ch * 64, h * dump_ld + it.key_lo + j * BN, bars.k_full(s));
                }
                ++ic;
            }
            if (!ok) {
                // give copies that are still in flight a bounded time to land before the CTA exits
                const long long t0 = clock64();
                for (int s = 0; s < S && kt > 0; ++s) {
                    const int last = kt - 1 - ((kt - 1 - s) % S + S) % S;  // last tile issued into stage s
                    if (last < 0) continue;
                    while (!ptx::mbar_try_wait(bars.k_full(s), (last / S) & 1) && clock64() - t0 < 40000000ll) {}
                }
            }
        }
    } else if (warp >= NEPI + 1 && warp <= NEPI + NISS) {
        // ------------------------------------------------------------------ MMA issuers
        // The (key tile, query tile) pairs of the CTA form one sequence; pair number q uses
        // accumulator buffer q mod 4, so the issue side runs up to four pairs ahead of the slowest
        // selection warp group.  Two threads in two warps take the pairs alternately, so the
        // barrier waits and the commit of one overlap with the MMAs of the other; a buffer is always
        // filled by the same issuer.  The commit after a pair's MMAs tells that pair's selection
        // warps that the scores are ready.  It goes to a barrier of its own per (buffer, query
        // tile): with three query tiles a warp group meets a buffer only every third time it is
        // filled, and a parity wait is sound only on a barrier whose every phase the waiter sees.
        if (lane == 0) {
            const int mine = warp - (NEPI + 1);
            // operand descriptors: the query tiles stay put, the key stages differ only in the start address
            uint64_t desc_q[NQT][Sh::KSTEPS], desc_k0[Sh::KSTEPS];
#pragma unroll
            for (int ks = 0; ks < Sh::KSTEPS; ++ks) {
                const int off = (ks / Sh::STEPS_PER_CH) * Sh::CH_BYTES + (ks % Sh::STEPS_PER_CH) * 32;
#pragma unroll
                for (int qt = 0; qt < NQT; ++qt) desc_q[qt][ks] = make_smem_desc<D>(ptx::smem_u32(sQ + qt * Sh::TILE_BYTES + off));
                desc_k0[ks] = make_smem_desc<D>(ptx::smem_u32(sK + off));
            }
            int kt = 0, ic = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < n_units; w += gridDim.x) {
                int h_unused;
                WorkItem it;
                if (!unit(w, h_unused, it)) continue;
                const int nq = (it.nrows + BM - 1) / BM;  // query tiles of the item that hold rows
                if (!(ok = wait_or_abort<0>(bars.q_full(), ic & 1, sAbort, sb, 3, wait_limit))) break;
                ptx::tc_fence_after();
                const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
                for (int j = 0; ok && (PRUNE || j < ntiles); ++j, ++kt) {
                    const int s = kt % S;
                    const uint64_t stage_off = (uint64_t)((s * Sh::TILE_BYTES) >> 4);  // start-address field counts 16-byte units
                    // Both issuers wait for EVERY key tile, also one whose pairs all belong to the other
                    // issuer (one query tile per CTA): a parity wait is sound only on a barrier whose
                    // every phase the waiter observes, and with an odd number of stages an issuer that
                    // skipped its partner's tiles would meet a stage only every second time it is filled.
                    if (!(ok = wait_or_abort<0>(bars.k_full(s), (kt / S) & 1, sAbort, sb, 4, wait_limit))) break;
                    int tile_key = 0, tile_dead = 0;
                    if constexpr (PRUNE) {
                        tile_key = sStageKey[s];
                        tile_dead = sStageDead[s];
                        ptx::mbar_arrive(bars.k_empty(s));  // the read is done: one of the arrivals the refill waits for
                    }
#pragma unroll
                    for (int qt = 0; qt < NQT; ++qt) {
                        const int seq = kt * NQT + qt;
                        if ((seq & 1) != mine) continue;
                        const int b = seq & (NBUF - 1);
                        if (!(ok = wait_or_abort<0>(bars.t_empty(b), ((seq >> 2) & 1) ^ 1, sAbort, sb, 5, wait_limit))) break;
                        ptx::tc_fence_after();
                        if constexpr (PRUNE) {
                            // a pair without scores (end of item, or ruled out for this query tile) still takes
                            // its turn in the ring, so that the buffers and barrier phases stay in step
                            const bool no_scores = tile_key == kEndOfItem || ((tile_dead >> qt) & 1);
                            sBufKey[b] = tile_key == kEndOfItem ? kEndOfItem : no_scores ? kDeadPair : tile_key;
                            __threadfence_block();
                            if (no_scores) {
                                ptx::mbar_arrive(bars.t_full(b, qt));
                                continue;
                            }
                        }
                        if (qt < nq) {
                            const uint32_t d_tmem = tmem_base + (uint32_t)(b * BN);
#pragma unroll
                            for (int ks = 0; ks < Sh::KSTEPS; ++ks)
                                ptx::mma_bf16_ss(d_tmem, desc_q[qt][ks], desc_k0[ks] + stage_off, kInstrDesc, ks > 0 ? 1u : 0u);
                        }
                        ptx::mma_commit(bars.t_full(b, qt));
                    }
                    if (PRUNE && ok && tile_key == kEndOfItem) {
                        ++kt;
                        break;
                    }
                }
                if (!ok) break;
                ptx::mma_commit(bars.q_empty());
                ++ic;
            }
            // all issued MMAs must have retired before tensor memory is released
            ptx::mma_commit(bars.done());
            const long long t0 = clock64();
            while (!ptx::mbar_try_wait(bars.done(), 0) && clock64() - t0 < 2000000000ll) {}
        }
    } else if (warp < NEPI) {
        // ------------------------------------------------------------------ selection warps
        const int qt = warp >> 2, quarter = warp & 3;
        cand_t* wblock = sRows + (size_t)(qt * 128 + quarter * 32) * Sp::SLOTS;  // this warp's block:
        uint32_t* wl = reinterpret_cast<uint32_t*>(wblock);                     // the lists (score plane, key plane) ...
        cand_t* wp = wblock + Sp::LIST * 32;                                    // ... then the pending slots
        const uint32_t wp_addr = ptx::smem_u32(wp + lane);                      // this lane's first pending slot
        const uint32_t wl_s = ptx::smem_u32(wl + lane);                         // this lane's list slot 0 (score plane)
        const uint32_t flush_req_s = ptx::smem_u32(const_cast<int*>(sFlushReq));
        const uint32_t full_bar0 = bars.t_full(0, qt);
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);  // buffer 0, this warp's lanes
        RowSel<KG> rs;
        int flush_seen = 0;
        int tcnt = 0, ic = 0;
        bool ok = true;
        for (long long w = blockIdx.x; ok && w < n_units; w += gridDim.x) {
            int h;
            WorkItem it;
            if (!unit(w, h, it)) continue;
            const bool active = qt * BM < it.nrows;  // an inactive query tile only keeps the barriers in step
            const int local = qt * BM + quarter * 32 + lane;
            const bool rvalid = local < it.nrows;
            if (active) row_init<KG>(rs, wl, k, lane, rvalid);
            __syncwarp();
            float inv_qn = 1.0f;
            if constexpr (PRUNE) {
                // nothing can be skipped for this warp's rows until a flush has raised their thresholds;
                // a warp without rows never objects
                if (active && rvalid) inv_qn = 1.0f / fmaxf(__ldg(pr.qnorm + (size_t)(it.row0 + local) * H + h), 1e-30f);
                publish_thresholds(active ? rs.tau : CUDART_INF_F, inv_qn, ic, warp_stat_s + 16u * warp, lane);
            }
            const int ntiles = (it.key_hi - it.key_lo + BN - 1) / BN;
            // This warp group's (key tile, query tile) pair is number tcnt*NQT + qt of the CTA; its buffer
            // is that number mod 4, and the (buffer, query tile) barrier has been used tcnt >> kUseShift
            // times before (pairs between two uses: 12, 4, 4 for NQT = 3, 2, 1).
            constexpr int kUseShift = NQT == 2 ? 1 : 2;
            if (DUMP || !active) {
                // debug dump of the raw scores, or a query tile past the item's rows that only keeps
                // the barriers in step
                for (int j = 0; PRUNE || j < ntiles; ++j, ++tcnt) {
                    const int b = (tcnt * NQT + qt) & (NBUF - 1);
                    ok = wait_or_abort(full_bar0 + (uint32_t)b * (8u * NQT), (uint32_t)(tcnt >> kUseShift) & 1u, sAbort, sb,
                                       6, wait_limit);
                    ok = __all_sync(FULL, ok);
                    if (!ok) break;
                    const int tile_key = PRUNE ? sBufKey[b] : 0;
                    if (quarter == 0 && lane == 0) ptx::mbar_arrive(bars.k_empty(tcnt % S));
                    ptx::tc_fence_after();
                    if (DUMP && active) {
                        const uint32_t taddr = taddr0 + (uint32_t)(b * BN);
                        const int key0 = it.key_lo + j * BN;
                        const int ncol = min(BN, it.key_hi - key0);
#pragma unroll 1
                        for (int c = 0; c < BN / 32; ++c) {
                            uint32_t v[32];
                            ptx::tmem_ld_32x32_sync(taddr + c * 32, v);
                            if (rvalid)
#pragma unroll
                                for (int x = 0; x < 32; ++x)
                                    if (c * 32 + x < ncol)
                                        dump[((size_t)h * dump_ld + it.row0 + local) * dump_ld + key0 + c * 32 + x] = __uint_as_float(v[x]);
                        }
                    }
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));
                    if (PRUNE && tile_key == kEndOfItem) {
                        ++tcnt;
                        break;
                    }
                }
            } else if constexpr (LSE) {
                // running maximum and sum of 2^(c (s - m)) over all keys of the graph, 64 columns at a time
                const float c2 = 1.4426950408889634f * rsqrtf((float)D);
                float m_run = -CUDART_INF_F, l_run = 0.0f;
                for (int j = 0; j < ntiles; ++j, ++tcnt) {
                    const int b = (tcnt * NQT + qt) & (NBUF - 1);
                    ok = wait_or_abort(full_bar0 + (uint32_t)b * (8u * NQT), (uint32_t)(tcnt >> kUseShift) & 1u, sAbort, sb,
                                       6, wait_limit);
                    ok = __all_sync(FULL, ok);
                    if (!ok) break;
                    if (quarter == 0 && lane == 0) ptx::mbar_arrive(bars.k_empty(tcnt % S));
                    ptx::tc_fence_after();
                    const uint32_t taddr = taddr0 + (uint32_t)(b * BN);
                    const int ncol = it.key_hi - (it.key_lo + j * BN);  // columns that exist; below 128 only in the last tile
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
                        uint32_t v[64];
                        ptx::tmem_ld_32x64_sync(taddr + half * 64, v);
                        if (half == 1) {
                            ptx::tc_fence_before();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));
                        }
                        if (ncol < BN) {
#pragma unroll
                            for (int x = 0; x < 64; ++x)
                                if (half * 64 + x >= ncol) v[x] = 0xFF800000u;  // -inf
                        }
                        float hm[8];
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const int o = 8 * g;
                            const float a0 = ptx::max3(__uint_as_float(v[o]), __uint_as_float(v[o + 1]), __uint_as_float(v[o + 2]));
                            const float a1 = ptx::max3(__uint_as_float(v[o + 3]), __uint_as_float(v[o + 4]), __uint_as_float(v[o + 5]));
                            hm[g] = ptx::max3(a0, a1, fmaxf(__uint_as_float(v[o + 6]), __uint_as_float(v[o + 7])));
                        }
                        const float tm = fmaxf(ptx::max3(hm[0], hm[1], hm[2]), ptx::max3(hm[3], hm[4], ptx::max3(hm[5], hm[6], hm[7])));
                        const float m_new = fmaxf(m_run, tm);
                        if (m_new > -CUDART_INF_F) {  // false only while every column so far was past the key range
                            const float off = -m_new * c2;
                            float add[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                            for (int x = 0; x < 64; ++x) add[x & 3] += ptx::ex2(fmaf(__uint_as_float(v[x]), c2, off));
                            l_run = l_run * ptx::ex2(fmaf(m_run, c2, off)) + ((add[0] + add[1]) + (add[2] + add[3]));
                            m_run = m_new;
                        }
                    }
                }
                if (ok && rvalid) {
                    const size_t o = (size_t)(it.row0 + local) * H + h;
                    const float* sc = topk_score + o * k;
                    float top = 0.0f;
                    for (int t = 0; t < k; ++t) {
                        const float x = __ldg(sc + t);
                        if (x > -CUDART_INF_F) top += ptx::ex2((x - m_run) * c2);
                    }
                    dump[o] = l_run > 0.0f ? fminf(top / l_run, 1.0f) : 0.0f;
                }
            } else {
                const int ragged_j = ((it.key_hi - it.key_lo) & (BN - 1)) ? ntiles - 1 : -1;  // only the last tile can be short
                int key0 = it.key_lo;
                for (int j = 0; PRUNE || j < ntiles; ++j, ++tcnt, key0 += BN) {
                    const int b = (tcnt * NQT + qt) & (NBUF - 1);
                    const uint32_t full_bar = full_bar0 + (uint32_t)b * (8u * NQT);
                    const uint32_t full_par = (uint32_t)(tcnt >> kUseShift) & 1u;
                    if (!__all_sync(FULL, ptx::mbar_try_wait(full_bar, full_par))) {
                        // The scores are still not there after the try's own (hardware-bounded) wait:
                        // merge pending candidates into the lists meanwhile (always allowed, and it
                        // raises the thresholds early), then block.
                        if (__any_sync(FULL, rs.cnt > 0)) {
                            flush_pending<KG>(rs, wl_s, wp_addr, rvalid);
                            if constexpr (PRUNE) publish_thresholds(rs.tau, inv_qn, ic, warp_stat_s + 16u * warp, lane);
                        }
                        ok = wait_or_abort(full_bar, full_par, sAbort, sb, 6, wait_limit);
                        ok = __all_sync(FULL, ok);
                        if (!ok) break;
                    }
                    if constexpr (PRUNE) key0 = sBufKey[b];  // the tiles that arrive are not consecutive
                    // this query tile's MMAs on the key tile have retired; once that holds for every query
                    // tile the key stage can be refilled
                    if (quarter == 0 && lane == 0) ptx::mbar_arrive(bars.k_empty(tcnt % S));
                    if (PRUNE && key0 < 0) {
                        __syncwarp();  // every lane has read the buffer's key
                        if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));
                        if (key0 == kDeadPair) continue;  // no scores for this query tile; the next pair follows
                        ++tcnt;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t taddr = taddr0 + (uint32_t)(b * BN);
                    const bool ragged = PRUNE ? key0 + BN > it.key_hi : j == ragged_j;
                    const int ncol = it.key_hi - key0;  // columns that exist; below 128 only in a ragged tile
                    // two 64-column halves keep the register footprint small; the accumulator buffer
                    // goes back to the MMA issuers as soon as the second half is in registers
                    float sub[16], quad[4];
                    uint32_t v[64];
                    ptx::tmem_ld_32x64_sync(taddr, v);
                    if (ragged) half_maxima<true>(v, ncol, sub, quad);
                    else half_maxima<false>(v, BN, sub, quad);
                    ptx::tmem_ld_32x64_sync(taddr + 64, v);
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bars.t_empty(b));
                    if (ragged) half_maxima<true>(v, ncol - 64, sub + 8, quad + 2);
                    else half_maxima<false>(v, BN, sub + 8, quad + 2);
                    const float gm = fmaxf(fmaxf(quad[0], quad[1]), fmaxf(quad[2], quad[3]));
                    // A flush by one warp stalls the others within a few tiles (the accumulator ring
                    // is only four deep), so the warps flush together: whoever must flush bumps a
                    // CTA-wide counter and every warp that sees it move flushes at its next tile.
                    const int req = (int)ptx::lds_u32(flush_req_s);
                    bool do_flush = req != flush_seen;
                    if (__any_sync(FULL, gm > rs.tau)) {  // some lane of the warp has a hit in this tile
                        uint32_t pend = wp_addr + (uint32_t)rs.cnt * 256u;
                        append_groups(sub, quad, rs.tau, key0, pend);
                        rs.cnt = (int)((pend - wp_addr) >> 8);
                        if (__any_sync(FULL, rs.cnt > ROOM - 16)) {  // a tile adds at most 16 groups per row
                            do_flush = true;
                            if (lane == 0 && req == flush_seen) atomicAdd(const_cast<int*>(sFlushReq), 1);
                        }
                    }
                    if (do_flush) {
                        flush_pending<KG>(rs, wl_s, wp_addr, rvalid);
                        if constexpr (PRUNE) publish_thresholds(rs.tau, inv_qn, ic, warp_stat_s + 16u * warp, lane);
                        flush_seen = req + ((req == flush_seen) ? 1 : 0);
                    }
                }
            }
            if (!ok) break;
            if (!DUMP && !LSE && active) {
                // finalise: drain the pending slots, then store each row's k groups (first key and
                // group maximum, unsorted; empty slots as -1 / -inf) for the rescoring kernel
                flush_pending<KG>(rs, wl_s, wp_addr, rvalid);
                __syncwarp();
                const int nloc = min(32, it.nrows - (qt * BM + quarter * 32));
                for (int r = 0; r < nloc; ++r) {
                    const int srow = it.row0 + qt * BM + quarter * 32 + r;  // sweep order; the result goes to the row's own place
                    const size_t o = ((size_t)(perm ? __ldg(perm + srow) : srow) * H + h) * k;
                    for (int t = lane; t < k; t += 32) {
                        const uint32_t c = wl[t * 32 + r];
                        topk_idx[o + t] = c ? (int)wl[Sp::LIST * 32 + t * 32 + r] : -1;
                        topk_score[o + t] = c ? unorder_bits(c) : -CUDART_INF_F;
                    }
                }
                __syncwarp();
            }
            ++ic;
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

// Tensor map over a bf16 matrix of `rows` rows of `row_elems` elements; a box is 128 rows x one
// swizzle span of columns.  Q is [N, H*d] (a head is a column block); the regrouped keys are
// [H*N, d] (a head is a row block, so a key tile is one contiguous piece of memory).
template <int D>
bool make_tensor_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t row_elems) {
    using Sh = TcShape<D>;
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)row_elems, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)row_elems * 2};
    const cuuint32_t box[2] = {(cuuint32_t)Sh::BOX_INNER, 128u};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUtensorMapSwizzle sw = Sh::SWB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : Sh::SWB == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int KG, int NQT, int S, bool DUMP, bool PRUNE, bool LSE = false>
cudaError_t launch_cfg(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    using Sh = TcShape<D>;
    using Sp = SmemPlan<KG, NQT, S>;
    constexpr size_t smem_bytes = 1024 + (size_t)(NQT + S) * Sh::TILE_BYTES + (size_t)NQT * 128 * Sp::SLOTS * 8 +
                                  (size_t)Sp::NBARS * 8 + 16 + 240;
    static_assert(smem_bytes <= 232448, "shared memory budget of one CTA");
    CUtensorMap tmQ, tmK;
    if (!make_tensor_map<D>(&tmQ, w.reorder ? static_cast<const void*>(a.ws + w.qperm_off) : a.Q, a.N, (int64_t)a.H * D) ||
        !make_tensor_map<D>(&tmK, a.ws + w.kpack_off, a.N * a.H, D))
        return cudaErrorInvalidValue;
    auto kern = score_select_tc_kernel<D, KG, NQT, S, DUMP, PRUNE, LSE>;
    PruneArgs pr{nullptr, nullptr, nullptr};
    if (PRUNE)
        pr = PruneArgs{reinterpret_cast<const float*>(a.ws + w.qstat_off), reinterpret_cast<const float*>(a.ws + w.kstat_off),
                       reinterpret_cast<const float*>(a.ws + w.qnorm_off)};
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (err != cudaSuccess) return err;
    const long long max_total = (long long)w.max_items * a.H;
    const int grid = (int)std::min<long long>(sm_count(), max_total);
    kern<<<grid, NQT * 128 + 96, smem_bytes, a.stream>>>(
        tmQ, tmK, reinterpret_cast<const WorkItem*>(a.ws + w.items_off), reinterpret_cast<StatusBlock*>(a.ws),
        a.H, a.k, a.topk_idx, a.topk_score, dump, (int)a.N, a.wait_limit_cycles > 0 ? a.wait_limit_cycles : kDefaultWaitLimitCycles,
        a.drop_first_tile, (w.reorder && !DUMP) ? reinterpret_cast<const int*>(a.ws + w.perm_off) : nullptr, pr);
    return cudaGetLastError();
}

template <int D, bool DUMP, bool PRUNE>
cudaError_t launch_d(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    // (list groups KG, query tiles per CTA, key stages) by k and head width; shared memory decides
    if (a.k <= 32) {
        if constexpr (D <= 32) return launch_cfg<D, 4, 3, 4, DUMP, PRUNE>(a, w, dump);
        else if constexpr (D == 64) return launch_cfg<D, 4, 2, 3, DUMP, PRUNE>(a, w, dump);
        else return launch_cfg<D, 4, 1, 3, DUMP, PRUNE>(a, w, dump);
    }
    if (a.k <= 64) {
        if constexpr (D <= 32) return launch_cfg<D, 8, 2, 3, DUMP, PRUNE>(a, w, dump);
        else if constexpr (D == 64) return launch_cfg<D, 8, 1, 4, DUMP, PRUNE>(a, w, dump);
        else return launch_cfg<D, 8, 1, 3, DUMP, PRUNE>(a, w, dump);
    }
    if constexpr (D <= 64) return launch_cfg<D, 16, 1, 3, DUMP, PRUNE>(a, w, dump);
    else return cudaErrorNotSupported;
}

template <bool DUMP, bool PRUNE>
cudaError_t launch_any(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    switch (a.d) {
        case 16: return launch_d<16, DUMP, PRUNE>(a, w, dump);
        case 32: return launch_d<32, DUMP, PRUNE>(a, w, dump);
        case 64: return launch_d<64, DUMP, PRUNE>(a, w, dump);
        case 128: return launch_d<128, DUMP, PRUNE>(a, w, dump);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace

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

bool score_select_tc_supported(int32_t d, int32_t k) {
    if (d != 16 && d != 32 && d != 64 && d != 128) return false;
    if (k <= 64) return true;
    return k <= 128 && d <= 64;
}

int score_select_tc_rows_per_item(int32_t d, int32_t k) {  // 128 * query tiles per CTA of launch_d's choice
    if (k <= 32) return d <= 32 ? 384 : d == 64 ? 256 : 128;
    return (k <= 64 && d <= 32) ? 256 : 128;
}  // 128 * query tiles per CTA

cudaError_t launch_score_select_tc(const FwdArgs& a, const FwdWorkspace& w) {
    return w.prune ? launch_any<false, true>(a, w, nullptr) : launch_any<false, false>(a, w, nullptr);
}

// The softmax-share diagnostic on the tensor cores: mass[i,h] as float [N, H].  The workspace must hold the
// regrouped keys and work items of score_select_tc_rows_per_item(d, 1) rows; the rows keep their order.
cudaError_t launch_topk_mass_tc(const FwdArgs& a, const FwdWorkspace& w, float* mass) {
    switch (a.d) {
        case 16: return launch_cfg<16, 4, 3, 4, false, false, true>(a, w, mass);
        case 32: return launch_cfg<32, 4, 3, 4, false, false, true>(a, w, mass);
        case 64: return launch_cfg<64, 4, 2, 3, false, false, true>(a, w, mass);
        case 128: return launch_cfg<128, 4, 1, 3, false, false, true>(a, w, mass);
        default: return cudaErrorNotSupported;
    }
}

// Test hook: same TMA / tcgen05 pipeline, but the selection warps write every score of the tile to
// dump[h][i][j] (ld = N) instead of filtering.  Only for small single problems.
cudaError_t launch_score_dump_tc(const FwdArgs& a, const FwdWorkspace& w, float* dump) {
    return launch_any<true, false>(a, w, dump);
}

}  // namespace kmip
