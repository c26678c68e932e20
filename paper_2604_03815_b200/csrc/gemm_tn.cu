// Dense projections of the full attention layer (Eq. 2; Algorithm 1 "Require" line and line 8):
//   C[M, N] = scale * A[M, K] B[N, K]^T,   A, B bf16 row-major (K contiguous), fp32 accumulation,
// on the 5th-generation tensor cores: TMA -> 4-stage shared-memory ring (128-byte swizzle) ->
// tcgen05.mma (M 128 x N 128 x K 16, accumulators in tensor memory) -> four epilogue warps that read
// the accumulators and store bf16 or fp32.  Two ways to put several products into one launch:
// "batched" - up to three (B, C, scale) triples share A (the Q, K and V projections of X), one grid
// layer each - and "summed" - C = sum_i A_i B_i^T over up to three K segments (dX = dQ W_Q + dK W_K +
// dV W_V).  The epilogue can drop the rows or columns that belong to the zero padding of a head
// (index i of a padded axis is kept iff i % pad < real and lands at (i / pad) * real + i % pad), which
// is how weight gradients come out in the weights' own shape.
// One CTA per 128 x 128 output tile; ragged edges are zero-filled by TMA on the way in and masked
// on the way out.  Every wait is bounded (status word KMIP_ERR_TIMEOUT, clean return).
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

namespace kmip {

namespace {

constexpr int GM = 128, GN = 128, GK = 64, GS = 4;
constexpr int kTileBytes = 128 * GK * 2;  // one operand tile: 128 rows of 128 bytes
constexpr int kGemmThreads = 192;         // warp 0: TMA producer, warp 1: MMA issuer (owns TMEM), warps 2-5: epilogue
constexpr unsigned FULL = 0xFFFFFFFFu;

// K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t gemm_desc(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// fp32 accumulate, bf16 A and B, both K-major, M = 128, N = 128
constexpr uint32_t kGemmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GN >> 3) << 17) | ((uint32_t)(GM >> 4) << 24);

struct GemmOut {
    void* C[3];
    float scale[3];
    int ldc;                 // elements between output rows
    int row_pad, row_real;   // rows with (m % row_pad) >= row_real are padding and dropped (row_pad = 0: keep all)
    int col_pad, col_real;   // the same for columns
    int out_f32;             // 1: fp32 output, 0: bf16
    int n_kseg;              // summed mode: K segments (1 otherwise)
};

__device__ __forceinline__ int drop_padding(int i, int pad, int real) {
    if (pad <= 0) return i;
    const int r = i % pad;
    return r < real ? (i / pad) * real + r : -1;
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, const GemmOut out, int M,
               int N, int K, StatusBlock* __restrict__ sb, long long wait_limit) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + GS * kTileBytes;
    uint64_t* sBars = reinterpret_cast<uint64_t*>(sB + GS * kTileBytes);
    uint32_t* sTmem = reinterpret_cast<uint32_t*>(sBars + 2 * GS + 1);
    volatile int* sAbort = reinterpret_cast<volatile int*>(sTmem + 1);
    const uint32_t bar0 = ptx::smem_u32(sBars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (GS + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * GS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * GM, n0 = blockIdx.y * GN, z = blockIdx.z;
    const CUtensorMap* tmAs[3] = {&tmA0, &tmA1, &tmA2};
    const CUtensorMap* tmBs[3] = {&tmB0, &tmB1, &tmB2};
    const int nk_seg = (K + GK - 1) / GK;      // K blocks per segment
    const int nk = nk_seg * out.n_kseg;        // batched mode: one segment, operand pair chosen by the grid layer

    if (threadIdx.x == 0) {
        for (int s = 0; s < GS; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        ptx::mbar_init(acc_full, 1);
        *sAbort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) { ptx::tmem_alloc(ptx::smem_u32(sTmem), GN); ptx::tmem_relinquish(); }
    if (warp == 0 && lane == 0) { ptx::prefetch_tensormap(&tmA0); ptx::prefetch_tensormap(tmBs[z]); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *sTmem;
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % GS;
                if (!(ok = ptx::mbar_wait_bounded<0>(empty(s), ((kb / GS) & 1) ^ 1, sAbort, wait_limit))) break;
                const int seg = out.n_kseg > 1 ? kb / nk_seg : 0, kk = (kb - seg * nk_seg) * GK;
                ptx::mbar_arrive_expect_tx(full(s), 2 * kTileBytes);
                ptx::tma_load_2d(ptx::smem_u32(sA + s * kTileBytes), tmAs[seg], kk, m0, full(s));
                ptx::tma_load_2d(ptx::smem_u32(sB + s * kTileBytes), tmBs[out.n_kseg > 1 ? seg : z], kk, n0, full(s));
            }
            if (!ok) record_status(sb, KMIP_ERR_TIMEOUT, 21);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % GS;
                if (!(ok = ptx::mbar_wait_bounded<0>(full(s), (kb / GS) & 1, sAbort, wait_limit))) break;
                ptx::tc_fence_after();
                const uint64_t da = gemm_desc(ptx::smem_u32(sA + s * kTileBytes)), db = gemm_desc(ptx::smem_u32(sB + s * kTileBytes));
#pragma unroll
                for (int ks = 0; ks < GK / 16; ++ks)
                    ptx::mma_bf16_ss(tmem, da + (uint64_t)(ks * 2), db + (uint64_t)(ks * 2), kGemmIdesc, (kb > 0 || ks > 0) ? 1u : 0u);
                ptx::mma_commit(empty(s));  // the stage is free once these MMAs have read it
            }
            if (ok) ptx::mma_commit(acc_full);
            else record_status(sb, KMIP_ERR_TIMEOUT, 22);
        }
    } else {
        // epilogue: warp w reads the TMEM lanes of its sub-partition, 32 rows x 32 columns at a time
        const int quarter = warp & 3;
        ok = ptx::mbar_wait_bounded<0>(acc_full, 0, sAbort, wait_limit);
        ok = __all_sync(FULL, ok);
        if (ok) {
            ptx::tc_fence_after();
            const int row = m0 + quarter * 32 + lane;
            const int orow = row < M ? drop_padding(row, out.row_pad, out.row_real) : -1;
            const float scale = out.scale[z];
#pragma unroll 1
            for (int c0 = 0; c0 < GN; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32_sync(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
                if (orow >= 0) {
#pragma unroll
                    for (int x = 0; x < 32; ++x) {
                        const int n = n0 + c0 + x;
                        const int ocol = n < N ? drop_padding(n, out.col_pad, out.col_real) : -1;
                        if (ocol >= 0) {
                            const size_t o = (size_t)orow * out.ldc + ocol;
                            const float val = __uint_as_float(v[x]) * scale;
                            if (out.out_f32) static_cast<float*>(out.C[z])[o] = val;
                            else static_cast<__nv_bfloat16*>(out.C[z])[o] = __float2bfloat16_rn(val);
                        }
                    }
                }
            }
        } else if (lane == 0) {
            record_status(sb, KMIP_ERR_TIMEOUT, 23);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) { ptx::tc_fence_after(); ptx::tmem_dealloc(tmem, GN); }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn gemm_encode_fn() {
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

// bf16 matrix [rows, cols] with `ld` elements between rows; a box is 128 rows x 64 columns, out-of-range parts read as 0
bool gemm_tensor_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld) {
    EncodeTiledFn enc = gemm_encode_fn();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)GK, 128u};
    const cuuint32_t estr[2] = {1u, 1u};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// batched (n_kseg = 1): n_batch (B, C, scale) triples over A[0]; summed (n_kseg > 1, n_batch = 1): C[0] =
// scale[0] * sum_i A[i] B[i]^T.  lda / ldb: elements between rows (multiples of 8, 16-byte aligned bases).
cudaError_t launch_gemm_tn(const void* const* A, int lda, const void* const* B, int ldb, void* const* C, const float* scale,
                           int n_batch, int n_kseg, int M, int N, int K, int ldc, int row_pad, int row_real, int col_pad,
                           int col_real, bool out_f32, StatusBlock* sb, cudaStream_t stream) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    if (n_batch < 1 || n_batch > 3 || n_kseg < 1 || n_kseg > 3 || (n_batch > 1 && n_kseg > 1) || (lda & 7) || (ldb & 7) || !sb)
        return cudaErrorInvalidValue;
    CUtensorMap tmA[3], tmB[3];
    GemmOut out;
    const int n_b = n_kseg > 1 ? n_kseg : n_batch;
    for (int z = 0; z < 3; ++z) {
        const int za = z < n_kseg ? z : 0, zb = z < n_b ? z : 0, zc = z < n_batch ? z : 0;
        if (!gemm_tensor_map(&tmA[z], A[za], M, K, lda) || !gemm_tensor_map(&tmB[z], B[zb], N, K, ldb)) return cudaErrorInvalidValue;
        out.C[z] = C[zc];
        out.scale[z] = scale ? scale[zc] : 1.0f;
    }
    out.ldc = ldc;
    out.row_pad = row_pad; out.row_real = row_real;
    out.col_pad = col_pad; out.col_real = col_real;
    out.out_f32 = out_f32 ? 1 : 0;
    out.n_kseg = n_kseg;
    constexpr size_t smem = 1024 + 2 * GS * kTileBytes + (2 * GS + 1) * 8 + 64;
    cudaError_t err = cudaFuncSetAttribute(gemm_tn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    const dim3 grid((M + GM - 1) / GM, (N + GN - 1) / GN, n_batch);
    gemm_tn_kernel<<<grid, kGemmThreads, smem, stream>>>(tmA[0], tmA[1], tmA[2], tmB[0], tmB[1], tmB[2], out, M, N, K, sb,
                                                         kDefaultWaitLimitCycles);
    return cudaGetLastError();
}

}  // namespace kmip
