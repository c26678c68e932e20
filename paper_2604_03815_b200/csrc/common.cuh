// Shared declarations of the k-MIP attention kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kmip.h"

namespace kmip {

// ---------------------------------------------------------------------------------------------
// Workspace layout.  The first 256 bytes are the status block; everything else is carved by the
// host-side planners below with 256-byte alignment.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStatusBytes = 256;
constexpr size_t kAlign = 256;

// -DKMIP_CHECKS builds (libkmip_checks.so) stand in for a memory checker: every workspace region is
// preceded by a 256-byte canary block that a tail kernel verifies, and the kernels test the indices they
// are about to follow.  A failed test RECORDS KMIP_ERR_CHECK in the status word and skips the access;
// nothing traps.  Release builds compile all of it away.
#ifdef KMIP_CHECKS
constexpr bool kChecks = true;
#else
constexpr bool kChecks = false;
#endif
constexpr size_t kCanaryBytes = kChecks ? 256 : 0;
constexpr uint32_t kCanaryWord = 0xC0DEFACEu;
constexpr int kMaxCanaries = 24;

// Offsets of the canary blocks of a workspace (checks builds; n = 0 otherwise).
struct Canaries {
    size_t off[kMaxCanaries];
    int n = 0;
};

struct StatusBlock {
    int status;      // kmip_status_t recorded by the device (first error wins)
    int detail;      // where it happened (kernel-specific code)
    int n_items;     // forward: number of work items the plan kernel produced
    int n_long;      // backward: number of long key segments
    // pruned sweep: key tiles of all work items, tiles loaded (end-of-item markers included),
    // (key tile, query tile) pairs, pairs scored - summed over the CTAs (kmip_attn_sweep_counters)
    unsigned long long counters[4];
    int n_redo;      // forward, fp16 prefilter: rows the rescoring kernel sent to the exact kernel
    int reserved[51];
};
static_assert(sizeof(StatusBlock) == kStatusBytes, "status block size");

// One unit of work of the tensor-core score kernel: up to 384 consecutive query rows of one
// graph and that graph's key range (Eq. 1 restricted to the graph by the CSR offsets).
struct WorkItem {
    int row0;    // first query row
    int nrows;   // 1..384 (128 x the query tiles per CTA of the launched configuration)
    int key_lo;  // graph's first row
    int key_hi;  // one past the graph's last row
    int tile0;   // number of the graph's first 128-key tile in the per-tile statistics (pruned sweep)
};

__host__ __device__ inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

struct FwdWorkspace {
    size_t items_off;  // WorkItem[max_items]
    size_t kpack_off;  // [H, N, d], 2 bytes per element: K regrouped by head for the tensor-core sweeps (bf16, or
                       // scaled fp16 for the half-precision prefilter; 0 bytes without a tensor-core sweep)
    size_t qperm_off;  // [N, H, d], 2 bytes per element: Q in the sweep's row order (bf16, only when `reorder`;
                       // scaled fp16 whenever `f16`)
    size_t perm_off;   // int  [N]: original row of each sweep row
    size_t code_off;   // u16  [N]: locality codes of the query rows
    // pruned sweep only (all 0 bytes otherwise):
    size_t kperm_off;   // int   [N]: original key of each sweep position
    size_t kcode_off;   // u16   [N]: key codes (norm class, nearest pivot), by node
    size_t kcs_off;     // u16   [N]: the same in sweep order
    size_t knorm_off;   // float [N]: squared norm of the node's whole key vector
    size_t gmax_off;    // u32   [G]: bits of each graph's largest squared key norm
    size_t qnorm_off;   // float [N, H]: norm of each query row's head slice, in sweep order
    size_t qstat_off;   // float [max_items, 3, H, d+4]: centroid, radius, centroid norm of each item's 128-row query tiles
    size_t kstat_off;   // float [max_tiles, H, d+4]: centroid, radius, centroid norm, largest norm of each key tile
    // half-precision prefilter only (all 0 bytes otherwise):
    size_t f16stat_off;    // F16HeadStat [H]: per-head norm maxima
    size_t cand_word_off;  // u32 [N, H, list]: the groups each row kept (first key of the 16-key window, bit 31 = odd keys)
    size_t cand_half_off;  // u16 [N, H, list]: their fp16 maxima
    size_t redo_off;       // int [N * H]: (row, head) pairs the rescoring kernel hands to the exact kernel
    size_t total;
    int max_items;
    int max_tiles;
    int list;          // groups kept per row by the half-precision prefilter
    bool tc;           // a tensor-core sweep runs (bf16 storage and a supported (d, k))
    bool f16;          // ... namely the half-precision prefilter (score_select_f16.cu)
    bool reorder;      // the sweep runs the rows of large graphs in locality order (reorder.cu)
    bool prune;        // the sweep skips key tiles that cannot hold a candidate (prune.cu)
    Canaries canaries;
};

constexpr int64_t kReorderMinNodes = 32768;  // below this the extra launches cost more than they can save

bool score_select_tc_supported(int32_t d, int32_t k);
bool score_select_f16_supported(int32_t d, int32_t k);
int score_select_f16_list(int32_t k);
int score_select_f16_rows_per_item(int32_t k);
int score_select_f16x4_rows_per_item();

// Which sweep the plan is for: the one the mode selects, or one a test entry point asks for.
enum PlanVariant { kPlanByMode = 0, kPlanNoTensorCore = 1, kPlanTcFp32Acc = 2, kPlanTcFp16Acc = 3,
                   kPlanTcFp32AccInOrder = 4 /* fp32-accumulate sweep over the rows in their own order */ };

inline FwdWorkspace plan_fwd_workspace(int64_t N, int32_t G, int32_t H, int32_t d, int32_t k, int mode,
                                       int variant = kPlanByMode) {
    FwdWorkspace w;
    // start of the next region after one that ends at `end`; checks builds put a canary block in front of it
    auto region = [&w](size_t end) {
        const size_t c = align_up(end);
        if (kChecks && w.canaries.n < kMaxCanaries) w.canaries.off[w.canaries.n++] = c;
        return c + kCanaryBytes;
    };
    const int32_t g = G > 0 ? G : 1;
    w.tc = variant == kPlanByMode ? (mode != KMIP_FP32_EXACT && score_select_tc_supported(d, k))
                                  : variant != kPlanNoTensorCore;
    w.f16 = variant == kPlanByMode ? (w.tc && mode == KMIP_BF16_TC && score_select_f16_supported(d, k))
                                   : variant == kPlanTcFp16Acc;
    w.list = w.f16 ? score_select_f16_list(k) : 0;
    w.max_items = (int)(N / 128 + g + 1);
    w.items_off = region(kStatusBytes);
    w.kpack_off = region(w.items_off + sizeof(WorkItem) * (size_t)w.max_items);
    w.reorder = w.tc && N >= kReorderMinNodes && variant != kPlanTcFp32AccInOrder;
    w.qperm_off = region(w.kpack_off + (w.tc ? (size_t)N * H * d * 2 : 0));
    w.perm_off = region(w.qperm_off + ((w.reorder || w.f16) ? (size_t)N * H * d * 2 : 0));
    w.code_off = region(w.perm_off + (w.reorder ? (size_t)N * 4 : 0));
    w.prune = variant == kPlanByMode && mode == KMIP_BF16_TC_PRUNED && w.reorder;
    w.max_tiles = (int)(N / 128 + g + 2);  // tile0 of a graph = floor(first row / 128) + graph index
    const size_t p = w.prune ? 1 : 0, rec = (size_t)(d + 4) * 4;
    w.kperm_off = region(w.code_off + (w.reorder ? (size_t)N * 2 : 0));
    w.kcode_off = region(w.kperm_off + p * (size_t)N * 4);
    w.kcs_off = region(w.kcode_off + p * (size_t)N * 2);
    w.knorm_off = region(w.kcs_off + p * (size_t)N * 2);
    w.gmax_off = region(w.knorm_off + p * (size_t)N * 4);
    w.qnorm_off = region(w.gmax_off + p * (size_t)g * 4);
    w.qstat_off = region(w.qnorm_off + p * (size_t)N * H * 4);
    w.kstat_off = region(w.qstat_off + p * (size_t)w.max_items * 3 * H * rec);
    const size_t f = w.f16 ? 1 : 0, rows = (size_t)N * H;
    w.f16stat_off = region(w.kstat_off + p * (size_t)w.max_tiles * H * rec);
    w.cand_word_off = region(w.f16stat_off + f * 16 * (size_t)H);
    w.cand_half_off = region(w.cand_word_off + f * rows * w.list * 4);
    w.redo_off = region(w.cand_half_off + f * rows * w.list * 2);
    w.total = region(w.redo_off + f * rows * 4);  // checks builds: a last canary block behind the last region
    return w;
}

struct BwdWorkspace {
    size_t p_off;         // float [N*H*k]   softmax weights
    size_t ds_off;        // float [N*H*k]   score gradients
    size_t seg_off;       // int   [N*H+1]   start of each (key, head) hit list
    size_t cursor_off;    // int   [N*H]     hit counts, then fill cursors
    size_t pairs_off;     // int4  [N*H*k]   hit lists: records {query row, p, dS, (key, head) number}
    size_t tmp_off;       // int4  [N*H*k]   the other buffer of the radix passes that build them
    size_t table_off;     // int   [high digits][blocks]  digit counts per block of the first sorting step, then offsets
    size_t tblsum_off;    // int   block sums of the scan over that table
    size_t blocksum_off;  // int   [scan blocks]
    size_t long_off;      // int   [N*H]     ids of long segments
    size_t total;
    int scan_blocks;
    Canaries canaries;
};

constexpr int kScanItemsPerBlock = 4096;
// The hit lists are built by a stable two-step radix sort of the selected pairs by (key, head) number, so every
// list comes out ordered by query row whatever the timing.  First step: a block owns kRadixPerWarp consecutive
// pairs per warp and sorts them by the high digit in shared memory before it writes them out.
constexpr int kRadixPerWarp = 512;
constexpr int kRadixMaxBits = 12, kRadixMaxBins = 1 << kRadixMaxBits;
struct RadixPlan {
    int bits, lo_bits, hi_bits;  // of the numbers 0 .. rows (rows = "no key"): low and high digit
    bool sorted;                 // false: more than 2 * kRadixMaxBits bits or 2^31 pairs, unordered lists instead
    int warps;                   // per block of the first step
    long long blocks;            // blocks of the first step
    size_t bins_hi;
};
inline RadixPlan plan_radix(long long rows, long long pairs) {
    RadixPlan r;
    r.bits = 1;
    while ((1ll << r.bits) <= rows) ++r.bits;
    r.hi_bits = r.bits / 2 > 0 ? r.bits / 2 : 1;
    r.lo_bits = r.bits - r.hi_bits;
    r.sorted = r.bits <= 2 * kRadixMaxBits && pairs < (1ll << 31);
    r.warps = 8;
    const long long per_block = (long long)r.warps * kRadixPerWarp;
    r.blocks = r.sorted ? (pairs + per_block - 1) / per_block : 1;
    if (r.blocks < 1) r.blocks = 1;
    r.bins_hi = r.sorted ? ((size_t)1 << r.hi_bits) : 1;
    return r;
}

inline BwdWorkspace plan_bwd_workspace(int64_t N, int32_t H, int32_t k) {
    BwdWorkspace w;
    const size_t rows = (size_t)N * H, pairs = rows * (size_t)k;
    w.scan_blocks = (int)((rows + 1 + kScanItemsPerBlock - 1) / kScanItemsPerBlock);
    auto region = [&w](size_t end) {
        const size_t c = align_up(end);
        if (kChecks && w.canaries.n < kMaxCanaries) w.canaries.off[w.canaries.n++] = c;
        return c + kCanaryBytes;
    };
    size_t o = region(kStatusBytes);
    w.p_off = o;        o = region(o + 4 * pairs);
    w.ds_off = o;       o = region(o + 4 * pairs);
    w.seg_off = o;      o = region(o + 4 * (rows + 1));
    w.cursor_off = o;   o = region(o + 4 * (rows + 1));
    w.pairs_off = o;    o = region(o + 16 * pairs);
    w.tmp_off = o;      o = region(o + 16 * pairs);
    const RadixPlan rp = plan_radix((long long)rows, (long long)pairs);
    w.table_off = o;    o = region(o + 4 * rp.bins_hi * (size_t)rp.blocks);
    w.tblsum_off = o;   o = region(o + 4 * (rp.bins_hi * (size_t)rp.blocks / kScanItemsPerBlock + 2));
    w.blocksum_off = o; o = region(o + 4 * (size_t)(w.scan_blocks + 1));
    w.long_off = o;     o = region(o + 4 * rows);
    w.total = o;
    return w;
}

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
__device__ inline void record_status(StatusBlock* sb, int status, int detail) {
    if (atomicCAS(&sb->status, 0, status) == 0) sb->detail = detail;
}
// Checks builds: `cond` must hold before an index is followed; if it does not, the failure is recorded with
// `code` (which test, see the call sites) and the caller skips the access.  Release builds: always true, no code.
__device__ __forceinline__ bool kmip_check(bool cond, StatusBlock* sb, int code) {
    if (!kChecks) return true;
    if (!cond) record_status(sb, KMIP_ERR_CHECK, code);
    return cond;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;  // elements per 16-byte vector
    __device__ static inline float load(const float* p) { return __ldg(p); }
    __device__ static inline void store(float* p, float v) { *p = v; }
    __device__ static inline void load_vec(const float* p, float (&v)[4]) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    __device__ static inline void store_vec(float* p, const float (&v)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static inline float load(const __nv_bfloat16* p) {
        return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    __device__ static inline void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
    __device__ static inline void load_vec(const __nv_bfloat16* p, float (&v)[8]) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static inline void store_vec(__nv_bfloat16* p, const float (&v)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&b);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// ---------------------------------------------------------------------------------------------
// Kernel launchers (defined in the .cu files; all asynchronous on `stream`)
// ---------------------------------------------------------------------------------------------
struct FwdArgs {
    const void *Q, *K, *V;
    const int32_t* graph_offsets;  // may be null
    int32_t G;
    int64_t N;
    int32_t H, d, k;
    int mode;
    void* out;
    int32_t* topk_idx;
    float* topk_score;
    unsigned char* ws;
    cudaStream_t stream;
    float drop_p = 0.0f;             // attention dropout on the k weights (0 = none)
    unsigned long long seed = 0ull;  // of its counter-based draws
    // per-call test options (kmip_test.h); the public entry points leave the defaults
    long long wait_limit_cycles = 0;  // bound of every device-side wait in SM clocks; <= 0: kDefaultWaitLimitCycles
    int drop_first_tile = 0;          // leave one key tile of CTA 0 unloaded, so that the waits on it run out
    int fp32_path = 0;                // fp32 mode: 0 = sweep chosen by problem size, 1 = one warp per row, 2 = tiled
};

constexpr long long kDefaultWaitLimitCycles = 8000000000ll;  // about 4 s of SM clocks

struct BwdArgs {
    const void *Q, *K, *V, *d_out;
    int64_t N;
    int32_t H, d, k;
    int mode;
    const int32_t* topk_idx;
    const float* topk_score;
    void *dQ, *dK, *dV;
    unsigned char* ws;
    cudaStream_t stream;
    float drop_p = 0.0f;
    unsigned long long seed = 0ull;
};

// plan.cu, checks builds: write the canary blocks of a workspace / verify them (detail = 900 + block number)
cudaError_t launch_canary_fill(unsigned char* ws, const Canaries& c, cudaStream_t stream);
cudaError_t launch_canary_check(unsigned char* ws, const Canaries& c, cudaStream_t stream);
// plan.cu: validates the offsets and writes the work items of the tensor-core kernel
cudaError_t launch_plan(const FwdArgs& a, const FwdWorkspace& w, int rows_per_item);
// plan.cu: K [N, H, d] -> [H, N, d] so that a head's key tile is one contiguous block for TMA
cudaError_t launch_pack_keys(const FwdArgs& a, const FwdWorkspace& w);
// reorder.cu: locality codes, per-graph bucket sort, row-permuted copy of Q (after launch_plan)
cudaError_t launch_reorder_queries(const FwdArgs& a, const FwdWorkspace& w);
// reorder.cu, pruned sweep: keys of large graphs sorted by (norm class, locality code) and regrouped by
// head in that order (replaces launch_pack_keys; after launch_reorder_queries, which owns the code buffer first)
cudaError_t launch_reorder_keys(const FwdArgs& a, const FwdWorkspace& w);
// prune.cu: centroid / radius / norm statistics of every item's query rows and of every key tile
cudaError_t launch_prune_stats(const FwdArgs& a, const FwdWorkspace& w);
constexpr int kMinRowsToSort = 8192;  // smaller graphs keep their row and key order
// score_select_exact.cu: CUDA-core scores + running top-k, any supported (d, k), fp32 or bf16 storage
cudaError_t launch_score_select_exact(const FwdArgs& a);
int sm_count();  // multiprocessors of the current device (cached per device)
// score_select_tc.cu: tcgen05 scores + running top-k (bf16 storage); returns cudaErrorNotSupported
// when (d, k) is outside what the tensor-core kernel covers
int score_select_tc_rows_per_item(int32_t d, int32_t k);
cudaError_t launch_score_select_tc(const FwdArgs& a, const FwdWorkspace& w);
cudaError_t launch_score_dump_tc(const FwdArgs& a, const FwdWorkspace& w, float* dump);
// Half-precision prefilter of the tensor-core mode, head widths 16 and 32, k <= 32:
// f16_convert.cu (norm maxima, scaled fp16 copies of K and Q), score_select_f16.cu (sweep: 384-row work items),
// refine_f16.cu (exact rescoring, redo list), score_select_exact.cu (the listed rows again, from all keys)
cudaError_t launch_f16_convert(const FwdArgs& a, const FwdWorkspace& w);
cudaError_t launch_score_select_f16(const FwdArgs& a, const FwdWorkspace& w);
cudaError_t launch_score_select_f16x4(const FwdArgs& a, const FwdWorkspace& w);  // k <= 16, called by the above
cudaError_t launch_score_dump_f16(const FwdArgs& a, const FwdWorkspace& w, float* dump);
cudaError_t launch_refine_f16(const FwdArgs& a, const FwdWorkspace& w);
cudaError_t launch_score_select_exact_redo(const FwdArgs& a, const FwdWorkspace& w);
// refine.cu: rescoring of the k best 8-key groups left by the tensor-core sweep -> final top-k
cudaError_t launch_refine_topk(const FwdArgs& a, const FwdWorkspace& w);
cudaError_t launch_refine_topk_fp32(const FwdArgs& a);
// topk_mass.cu: share of the full softmax held by the kept scores on CUDA cores (fp32 storage); needs 128-row
// work items in the workspace.  score_select_tc.cu: the same on the tensor cores (bf16 storage, every head width)
cudaError_t launch_topk_mass(const FwdArgs& a, const FwdWorkspace& w, float* mass);
cudaError_t launch_topk_mass_tc(const FwdArgs& a, const FwdWorkspace& w, float* mass);
// tiled CUDA-core sweep of fp32 mode (score_select_fp32.cu): 128-row work items, then launch_refine_topk_fp32
bool score_select_fp32_tiled_supported(int32_t d, int32_t k);
cudaError_t launch_score_select_fp32_tiled(const FwdArgs& a, const FwdWorkspace& w);
// epilogue.cu: softmax over the k kept scores fused with the gather-V weighted sum
cudaError_t launch_softmax_gather(const FwdArgs& a);
// backward.cu
// ev (optional): three events recorded after the rows, inverse-index and segment stages
cudaError_t launch_backward(const BwdArgs& a, const BwdWorkspace& w, cudaEvent_t* ev);

// gemm_tn.cu: C = scale * A B^T on the tensor cores (bf16 operands with K contiguous, fp32 accumulation); see there
cudaError_t launch_gemm_tn(const void* const* A, int lda, const void* const* B, int ldb, void* const* C, const float* scale,
                           int n_batch, int n_kseg, int M, int N, int K, int ldc, int row_pad, int row_real, int col_pad,
                           int col_real, bool out_f32, StatusBlock* sb, cudaStream_t stream);

// layer.cu: the full layer of Eq. 2 (bf16).  All pointers are device memory.
struct LayerArgs {
    const void *x, *w_q, *w_k, *w_v, *w_o;  // [N, d_model], [H*d_head, d_model] x 3, [d_model, H*d_head]
    void *q, *k_proj, *v, *o;               // [N, H, d_pad]: written by the forward pass, read by the backward pass
    int32_t* topk_idx;                      // [N, H, k]
    float* topk_score;                      // [N, H, k]
    void* y;                                // forward: [N, d_model]
    const void* d_y;                        // backward: upstream gradient [N, d_model]
    void *d_x, *dw_q, *dw_k, *dw_v, *dw_o;  // backward: gradients in the shapes of x and the weights
    const int32_t* graph_offsets;
    int32_t G;
    int64_t N;
    int32_t d_model, H, d_head, k;
    unsigned char* ws;
    cudaStream_t stream;
};
struct LayerWorkspace {
    size_t wq_pad, wk_pad, wv_pad, wo_pad;         // padded weights
    size_t wqT, wkT, wvT, woT;                     // their transposes (backward)
    size_t d_o, d_q, d_k, d_v;                     // [N, H*d_pad] gradients around the attention core
    size_t xT, dyT, oT, dqT, dkT, dvT;             // transposed activations for the weight gradients
    size_t attn, attn_bytes;                       // workspace of the attention call
    size_t total;
};
int layer_pad_width(int d_head);
LayerWorkspace plan_layer_workspace(int64_t N, int32_t G, int32_t d_model, int32_t H, int32_t d_head, int32_t k, int pass);
int layer_forward(const LayerArgs& a);   // kmip_status_t
int layer_backward(const LayerArgs& a);

}  // namespace kmip
