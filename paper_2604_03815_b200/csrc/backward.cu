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

        // dP_t = g_i . v_{j_t}
        float dP[kMaxEntriesPerLane];
        gather_dot<T, D>(V, H, h, k, lane, dOut + (size_t)r * D, j, dP);
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

// In-place exclusive scan of n ints given the scanned sums of its 4096-item blocks (scan_block_sums_kernel,
// scan_block_offsets_kernel).
__global__ void __launch_bounds__(kScanThreads)
scan_inplace_kernel(int* __restrict__ v, long long n, const int* __restrict__ block_sums) {
    __shared__ int s_warp[32];
    const long long base = (long long)blockIdx.x * kScanItemsPerBlock + (long long)threadIdx.x * kScanPerThread;
    int c[kScanPerThread];
    int t = 0;
#pragma unroll
    for (int u = 0; u < kScanPerThread; ++u) {
        c[u] = (base + u < n) ? v[base + u] : 0;
        t += c[u];
    }
    int total;
    int off = block_sums[blockIdx.x] + block_exclusive_scan_1024(t, s_warp, total);
#pragma unroll
    for (int u = 0; u < kScanPerThread; ++u) {
        if (base + u < n) v[base + u] = off;
        off += c[u];
    }
}

// ---- hit lists by a stable radix sort --------------------------------------------------------------
// A hit record is everything the segment reduction needs about one selected pair in one 16-byte load:
// {query row, softmax weight p (times the dropout factor), score gradient dS, (key, head) number}.
// The records are sorted by (key, head) number in two stable steps, and the pairs start out in query
// order, so each key's list ends up ordered by query row - the same order on every run, which makes the
// sums of the segment stage reproducible bit for bit.  Pairs without a key (padding slots) get the number
// n_rows and sort behind every list.
//   partition  by the high digit of the number into buckets of 2^lo consecutive numbers.  A block owns a
//              contiguous range of the pairs (512 per warp).  A first kernel counts the digits of every block;
//              an exclusive scan over (digit, block) gives every block the place where its records of a digit
//              start.  The second kernel sorts the block's records by digit inside shared memory - each warp
//              counts the digits of its part, the counts are prefix-summed over the warps and the digits,
//              and each warp walks its part again, 32 records at a time, ranking equal digits by lane with a
//              match vote and advancing its own offsets - and then copies the sorted block out, so that the
//              records of a digit leave as one contiguous run.  No atomics decide a position: nothing depends
//              on timing.
//   buckets    one block per bucket sorts its records (a few hundred KB, served by L2) by the low digit
//              with the same count / scan / ranked walk, its eight warps owning contiguous parts.
struct RadixSrc {
    const int32_t* topk_idx;
    const float* ws_p;
    const float* ws_ds;
    int N, H, k;
    int n_rows;
};

// Lanes of the warp whose digit equals this lane's; lanes that hold no record vote with values of their own,
// which match nobody.
__device__ __forceinline__ unsigned warp_same_digit(int digit, bool live) {
    return __match_any_sync(0xFFFFFFFFu, live ? digit : (1 << kRadixMaxBits) + (int)(threadIdx.x & 31));
}

__device__ __forceinline__ int radix_key(const RadixSrc& s, long long e, int j) {
    return (j >= 0 && j < s.N) ? j * s.H + (int)((e / s.k) % s.H) : s.n_rows;
}

// table[digit][block] = number of the block's pairs with that high digit
__global__ void __launch_bounds__(512)
radix_count_kernel(const RadixSrc src, long long n, int per_block, int shift, int bins, int n_blocks,
                   int* __restrict__ table, StatusBlock* __restrict__ sb) {
    extern __shared__ unsigned s_hist[];  // [bins]
    for (int x = threadIdx.x; x < bins; x += blockDim.x) s_hist[x] = 0u;
    __syncthreads();
    const long long lo = (long long)blockIdx.x * per_block, hi = min(n, lo + per_block);
    for (long long e = lo + threadIdx.x; e < hi; e += blockDim.x) {
        const int j = __ldg(src.topk_idx + e);
        kmip_check(j < src.N, sb, 105);  // checks builds: an index the forward pass cannot have written (ignored either way)
        atomicAdd(s_hist + ((radix_key(src, e, j) >> shift) & (bins - 1)), 1u);  // shared memory; the counts do not depend on the order
    }
    __syncthreads();
    for (int d = threadIdx.x; d < bins; d += blockDim.x) table[(size_t)d * n_blocks + blockIdx.x] = (int)s_hist[d];
}

// table: after the scan, table[digit][block] is where the block's records of that digit start in dst.
// Shared memory: the block's records [warps * 512] (16 bytes each), per-warp digit counters (16 bits, [warps][bins]),
// where each digit starts inside the block (16 bits, [bins]) and in dst (32 bits, [bins]).
__global__ void __launch_bounds__(512)
radix_scatter_kernel(const RadixSrc src, long long n, int shift, int bins, int n_blocks, const int* __restrict__ table,
                     int4* __restrict__ dst, StatusBlock* __restrict__ sb) {
    extern __shared__ int4 s_rec[];
    const int warps = blockDim.x >> 5, per_block = warps * kRadixPerWarp;
    unsigned short* s_cnt = reinterpret_cast<unsigned short*>(s_rec + per_block);
    unsigned short* s_dstart = s_cnt + warps * bins;
    int* s_base = reinterpret_cast<int*>(s_dstart + bins);
    __shared__ int s_scan[16];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int x = threadIdx.x; x < warps * bins / 2; x += blockDim.x) reinterpret_cast<unsigned*>(s_cnt)[x] = 0u;
    for (int d = threadIdx.x; d < bins; d += blockDim.x) s_base[d] = __ldg(table + (size_t)d * n_blocks + blockIdx.x);
    __syncthreads();
    const long long lo = (long long)blockIdx.x * per_block + (long long)w * kRadixPerWarp;
    const long long hi = min(n, lo + kRadixPerWarp);
    constexpr int R = kRadixPerWarp / 32;  // rounds of 32 pairs per warp
    int key[R];
    float pw[R], dsw[R];  // everything the block reads from memory is requested here, before any of it is used
    unsigned short* cnt = s_cnt + w * bins;
#pragma unroll
    for (int u = 0; u < R; ++u) {
        const long long e = lo + u * 32 + lane;
        key[u] = e < hi ? __ldg(src.topk_idx + e) : -1;
        pw[u] = e < hi ? __ldg(src.ws_p + e) : 0.0f;
        dsw[u] = e < hi ? __ldg(src.ws_ds + e) : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < R; ++u) {
        const long long e = lo + u * 32 + lane;
        key[u] = e < hi ? radix_key(src, e, key[u]) : -1;
    }
    // the warp's digit counts (two 16-bit counters to a word; shared-memory atomics: counts do not depend on the order)
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int u = 0; u < R; ++u) {
        if (key[u] >= 0) {
            const int digit = (key[u] >> shift) & (bins - 1);
            atomicAdd(reinterpret_cast<unsigned*>(cnt) + (digit >> 1), 1u << (16 * (digit & 1)));
        }
    }
    __syncthreads();
    // counts -> offsets: per digit over the warps, then over the digits (each thread owns DPT consecutive digits)
    {
        const int DPT = (bins + (int)blockDim.x - 1) / (int)blockDim.x;
        const int d0 = threadIdx.x * DPT;
        int mine = 0;
        for (int i = 0; i < DPT; ++i) {
            const int d = d0 + i;
            if (d >= bins) break;
            int c[16];
#pragma unroll
            for (int ww = 0; ww < 16; ++ww) c[ww] = ww < warps ? s_cnt[ww * bins + d] : 0;
            int run = 0;
#pragma unroll
            for (int ww = 0; ww < 16; ++ww) {
                if (ww < warps) s_cnt[ww * bins + d] = (unsigned short)run;
                run += c[ww];
            }
            s_dstart[d] = (unsigned short)run;  // the digit's total for now
            mine += run;
        }
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_scan[w] = incl;
        __syncthreads();
        if (w == 0) {
            int v = lane < warps ? s_scan[lane] : 0;
#pragma unroll
            for (int o = 1; o < 16; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, v, o);
                if (lane >= o) v += t;
            }
            if (lane < warps) s_scan[lane] = v;
        }
        __syncthreads();
        int run = (w ? s_scan[w - 1] : 0) + incl - mine;
        for (int i = 0; i < DPT; ++i) {
            const int d = d0 + i;
            if (d >= bins) break;
            const int c = s_dstart[d];
            s_dstart[d] = (unsigned short)run;
            run += c;
        }
    }
    __syncthreads();
    // ranked walk into the block's sorted order
#pragma unroll
    for (int u = 0; u < R; ++u) {
        const long long e = lo + u * 32 + lane;
        const bool live = key[u] >= 0;
        int4 rec = make_int4(0, 0, 0, 0);
        if (live) {
            const long long r = e / src.k;  // query * H + head
            rec = make_int4((int)(r / src.H), __float_as_int(pw[u]), __float_as_int(dsw[u]), key[u]);
        }
        const int digit = (key[u] >> shift) & (bins - 1);
        const unsigned same = warp_same_digit(digit, live);
        if (live) {
            const int placed = cnt[digit];
            s_rec[s_dstart[digit] + placed + __popc(same & lt)] = rec;
            __syncwarp(same);
            if ((same & lt) == 0u) cnt[digit] = (unsigned short)(placed + __popc(same));  // the group's first lane moves the digit on
        }
        __syncwarp();
    }
    __syncthreads();
    const int total = (int)min((long long)per_block, n - (long long)blockIdx.x * per_block);
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int4 rec = s_rec[i];
        const int digit = (rec.w >> shift) & (bins - 1);
        const long long pos = (long long)s_base[digit] + (i - (int)s_dstart[digit]);
        if (kmip_check(pos >= 0 && pos < n, sb, 104)) dst[pos] = rec;  // checks builds: inside the buffer
    }
}

// Fallback beyond 2^24 (node, head) pairs, where the two-digit sort above would need tables of more than
// 4096 digits: every pair takes the next free place of its list with an atomic counter.  The lists then hold
// the same records in an order that depends on timing, so dK and dV are reproducible to fp32 rounding only.
__global__ void fill_unordered_kernel(const int32_t* __restrict__ topk_idx, long long n_pairs, int N, int H, int k,
                                      const float* __restrict__ ws_p, const float* __restrict__ ws_ds,
                                      const int* __restrict__ seg_off, int* __restrict__ cursor, int4* __restrict__ hits,
                                      StatusBlock* __restrict__ sb) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_pairs) return;
    const int j = __ldg(topk_idx + e);
    if (j < 0 || j >= N) return;
    const long long r = e / k;  // query * H + head
    const size_t key = (size_t)j * H + (int)(r % H);
    const long long pos = (long long)seg_off[key] + atomicAdd(cursor + key, 1);
    if (!kmip_check(pos >= 0 && pos < n_pairs, sb, 104)) return;  // checks builds: inside the hit lists
    hits[pos] = make_int4((int)(r / H), __float_as_int(__ldg(ws_p + e)), __float_as_int(__ldg(ws_ds + e)), (int)key);
}

// Second step: the records of one bucket (high digit = blockIdx.x), src -> dst, ordered by the low digit and,
// within a digit, in the order they have in src.  bucket_start[d * start_stride] is where bucket d begins.  The low
// digit of a number inside its bucket IS the (key, head) pair, so this kernel also knows where every list starts:
// it writes seg_off (rows + 1 entries) and the list of long segments.
constexpr int kBucketWarps = 8;
__global__ void __launch_bounds__(kBucketWarps * 32)
radix_bucket_kernel(const int4* __restrict__ src, int4* __restrict__ dst, const int* __restrict__ bucket_start, int start_stride, int n_buckets,
                    long long n, int lo_bits, long long n_rows, int* __restrict__ seg_off, int* __restrict__ long_list,
                    StatusBlock* __restrict__ sb) {
    extern __shared__ int s_cnt[];  // [kBucketWarps][bins]: counts, then next free positions
    __shared__ int s_tot[32];
    __shared__ int s_carry;
    const int bins = 1 << lo_bits;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d_hi = blockIdx.x;
    const long long begin = bucket_start[(size_t)d_hi * start_stride];
    const long long end = d_hi + 1 < n_buckets ? (long long)bucket_start[(size_t)(d_hi + 1) * start_stride] : n;
    const long long len = end - begin;
    for (int x = threadIdx.x; x < kBucketWarps * bins; x += blockDim.x) s_cnt[x] = 0;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    const long long per = ((len + kBucketWarps - 1) / kBucketWarps + 31) / 32 * 32;
    const long long lo = begin + (long long)w * per, hi = min(end, lo + per);
    int* cnt = s_cnt + w * bins;
    constexpr int U = 8;
    for (long long e0 = lo; e0 < hi; e0 += 32 * U) {
        int key[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long e = e0 + u * 32 + lane;
            key[u] = e < hi ? __ldg(reinterpret_cast<const int*>(src + e) + 3) : -1;
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (key[u] >= 0) atomicAdd(cnt + (key[u] & (bins - 1)), 1);  // shared memory; counts do not depend on the order
    }
    __syncthreads();
    // exclusive scan over (digit, warp): thread per digit across the warps, then the digit totals across the block
    for (int d0 = 0; d0 < bins; d0 += blockDim.x) {
        const int d = d0 + threadIdx.x;
        int tot = 0;
        if (d < bins) {
#pragma unroll
            for (int ww = 0; ww < kBucketWarps; ++ww) {
                const int c = s_cnt[ww * bins + d];
                s_cnt[ww * bins + d] = tot;  // warp ww's first record of this digit, relative to the digit's start
                tot += c;
            }
        }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_tot[w] = incl;
        __syncthreads();
        if (w == 0) {
            int v = lane < kBucketWarps ? s_tot[lane] : 0;
#pragma unroll
            for (int o = 1; o < kBucketWarps; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, v, o);
                if (lane >= o) v += t;
            }
            if (lane < kBucketWarps) s_tot[lane] = v;  // inclusive over warps
        }
        __syncthreads();
        const int digit_start = s_carry + (w ? s_tot[w - 1] : 0) + incl - tot;
        if (d < bins) {
#pragma unroll
            for (int ww = 0; ww < kBucketWarps; ++ww) s_cnt[ww * bins + d] += digit_start;
            // this digit is (key, head) pair number d_hi * bins + d: its list starts here and holds `tot` hits
            const long long pair = (long long)d_hi * bins + d;
            if (pair <= n_rows) seg_off[pair] = (int)(begin + digit_start);
            if (pair < n_rows && tot > kLongSeg) long_list[atomicAdd(&sb->n_long, 1)] = (int)pair;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_carry += s_tot[kBucketWarps - 1];
        __syncthreads();
    }
    // ranked walk, as in radix_scatter_kernel
    const unsigned lt = (1u << lane) - 1u;
    for (long long e0 = lo; e0 < hi; e0 += 32 * U) {
        int4 recs[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long e = e0 + u * 32 + lane;
            recs[u] = e < hi ? __ldg(src + e) : make_int4(0, 0, 0, -1);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (e0 + u * 32 >= hi) break;  // warp-uniform
            const int4 rec = recs[u];
            const bool live = e0 + u * 32 + lane < hi;
            const int digit = rec.w & (bins - 1);
            const unsigned same = warp_same_digit(digit, live);
            if (live) {
                const int base = cnt[digit];
                const long long pos = begin + base + __popc(same & lt);
                if (kmip_check(pos >= begin && pos < end, sb, 106)) dst[pos] = rec;  // checks builds: inside the bucket
                __syncwarp(same);
                if ((same & lt) == 0u) cnt[digit] = base + __popc(same);
            }
            __syncwarp();
        }
    }
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
    int4* tmp = reinterpret_cast<int4*>(a.ws + w.tmp_off);
    int* table = reinterpret_cast<int*>(a.ws + w.table_off);
    int* tblsum = reinterpret_cast<int*>(a.ws + w.tblsum_off);
    int* block_sums = reinterpret_cast<int*>(a.ws + w.blocksum_off);
    int* long_list = reinterpret_cast<int*>(a.ws + w.long_off);
    const T *Q = static_cast<const T*>(a.Q), *K = static_cast<const T*>(a.K), *V = static_cast<const T*>(a.V);
    const T* dOut = static_cast<const T*>(a.d_out);
    const float scale = 1.0f / sqrtf((float)a.d);
    cudaError_t err;

    const int row_blocks = (int)std::min<long long>((n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock, (long long)sm_count() * 32);
    bwd_rows_kernel<T, D><<<row_blocks, kWarpsPerBlock * 32, 0, a.stream>>>(
        K, V, dOut, a.topk_idx, a.topk_score, (int)a.N, a.H, a.k, scale, a.drop_p, a.seed, ws_p, ws_ds,
        static_cast<T*>(a.dQ));
    if (ev) cudaEventRecord(ev[0], a.stream);

    const int pair_blocks = (int)((n_pairs + 255) / 256);
    // the hit lists: stable partition of the pairs by the high digit of their (key, head) number, then a stable
    // sort of every bucket by the low digit, which also writes the list offsets
    {
        const RadixPlan rp = plan_radix(n_rows, n_pairs);
        if (!rp.sorted) {
            // more than 16.7 million (node, head) pairs or 2^31 selected pairs: unordered lists
            if ((err = cudaMemsetAsync(cursor, 0, sizeof(int) * (size_t)(n_rows + 1), a.stream)) != cudaSuccess) return err;
            hist_kernel<<<pair_blocks, 256, 0, a.stream>>>(a.topk_idx, n_pairs, (int)a.N, a.H, a.k, cursor, sb);
            scan_block_sums_kernel<<<w.scan_blocks, kScanThreads, 0, a.stream>>>(cursor, n_rows, block_sums);
            scan_block_offsets_kernel<<<1, kScanThreads, 0, a.stream>>>(block_sums, w.scan_blocks);
            scan_write_kernel<<<w.scan_blocks, kScanThreads, 0, a.stream>>>(cursor, n_rows, block_sums, seg_off, long_list, sb);
            fill_unordered_kernel<<<pair_blocks, 256, 0, a.stream>>>(a.topk_idx, n_pairs, (int)a.N, a.H, a.k, ws_p, ws_ds, seg_off,
                                                                    cursor, hits, sb);
        } else {
            const int bins_hi = 1 << rp.hi_bits, bins_lo = 1 << rp.lo_bits, n_blocks = (int)rp.blocks;
            const int per_block = rp.warps * kRadixPerWarp;
            const long long n_tab = (long long)bins_hi * n_blocks;
            const int tab_blocks = (int)((n_tab + kScanItemsPerBlock - 1) / kScanItemsPerBlock);
            const size_t smem_cnt = (size_t)bins_hi * sizeof(unsigned);
            const size_t smem_sct = (size_t)per_block * sizeof(int4) + (size_t)rp.warps * bins_hi * 2 + (size_t)bins_hi * 2 + (size_t)bins_hi * sizeof(int);
            const size_t smem_lo = (size_t)kBucketWarps * bins_lo * sizeof(int);
            if ((err = cudaFuncSetAttribute(radix_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_sct)) != cudaSuccess ||
                (err = cudaFuncSetAttribute(radix_bucket_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_lo)) != cudaSuccess)
                return err;
            RadixSrc src{a.topk_idx, ws_p, ws_ds, (int)a.N, a.H, a.k, (int)n_rows};
            radix_count_kernel<<<n_blocks, 512, smem_cnt, a.stream>>>(src, n_pairs, per_block, rp.lo_bits, bins_hi, n_blocks, table, sb);
            scan_block_sums_kernel<<<tab_blocks, kScanThreads, 0, a.stream>>>(table, n_tab, tblsum);
            scan_block_offsets_kernel<<<1, kScanThreads, 0, a.stream>>>(tblsum, tab_blocks);
            scan_inplace_kernel<<<tab_blocks, kScanThreads, 0, a.stream>>>(table, n_tab, tblsum);
            radix_scatter_kernel<<<n_blocks, rp.warps * 32, smem_sct, a.stream>>>(src, n_pairs, rp.lo_bits, bins_hi, n_blocks, table, tmp, sb);
            radix_bucket_kernel<<<bins_hi, kBucketWarps * 32, smem_lo, a.stream>>>(tmp, hits, table, n_blocks, bins_hi, n_pairs, rp.lo_bits, n_rows,
                                                                                seg_off, long_list, sb);
        }
    }
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
