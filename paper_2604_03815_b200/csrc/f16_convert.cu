// Operand copies of the half-precision prefilter sweep (score_select_f16.cu): per-head norm maxima,
// then K regrouped by head and Q in the sweep's row order, both scaled by a power of two per head and
// converted from bf16 to fp16.  bf16 has 8 significant bits and fp16 has 11, so the conversion of a
// scaled value is exact unless it falls below 2^-14 (fp16's smallest normal number), where it is
// rounded to a multiple of 2^-24; refine_f16.cu accounts for that in its error bound.
#include "common.cuh"
#include "f16_filter.cuh"

#include <cuda_fp16.h>

namespace kmip {

namespace {

template <int D>
__global__ void f16_norm_max_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                                    long long n_rows, int H, unsigned* __restrict__ stat,
                                    const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n_rows) return;
    const int h = (int)(r % H);
    float q2 = 0.0f, k2 = 0.0f, ka2 = 0.0f;
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 8) {
        float qv[8], kv[8];
        Elem<__nv_bfloat16>::load_vec(Q + r * D + c0, qv);
        Elem<__nv_bfloat16>::load_vec(K + r * D + c0, kv);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            q2 = fmaf(qv[c], qv[c], q2);
            k2 = fmaf(kv[c], kv[c], k2);
        }
        if (c0 == 8) ka2 = k2;
    }
    if (D == 16) ka2 = k2;
    // rounded up a little so that the fp32 sums above never understate a norm
    const unsigned vals[3] = {__float_as_uint(q2 * 1.00001f), __float_as_uint(k2 * 1.00001f), __float_as_uint(ka2 * 1.00001f)};
#pragma unroll
    for (int x = 0; x < 3; ++x)
        if (vals[x] > stat[h * 4 + x] && vals[x] < 0x7F800000u) atomicMax(stat + h * 4 + x, vals[x]);
}

__device__ __forceinline__ uint4 scale_to_half8(uint4 raw, float s) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2 h = __floats2half2_rn(__uint_as_float(w[i] << 16) * s, __uint_as_float(w[i] & 0xFFFF0000u) * s);
        o[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// K [N, H, d] bf16 -> [H, N, d] fp16, scaled per head; 16 bytes per thread.
__global__ void f16_convert_keys_kernel(const uint4* __restrict__ K, uint4* __restrict__ Kp, long long n_vec, int N, int H,
                                        int vec_per_row, const F16HeadStat* __restrict__ stat,
                                        const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const long long rowh = v / vec_per_row;  // j * H + h
    const int c = (int)(v % vec_per_row);
    const long long j = rowh / H;
    const int h = (int)(rowh % H);
    Kp[((long long)h * N + j) * vec_per_row + c] = scale_to_half8(__ldg(K + v), f16_scale_from_n2max(stat[h].k_n2max));
}

// Qp[p, :] = fp16(scale * Q[perm[p], :]) (perm == NULL: the identity); 16 bytes per thread.
__global__ void f16_convert_queries_kernel(const uint4* __restrict__ Q, const int* __restrict__ perm, uint4* __restrict__ Qp,
                                           long long n_vec, int vec_per_node, int vec_per_head,
                                           const F16HeadStat* __restrict__ stat, const StatusBlock* __restrict__ sb) {
    if (sb->status != KMIP_OK) return;
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const long long p = v / vec_per_node;
    const int c = (int)(v % vec_per_node);
    const long long src = perm ? (long long)__ldg(perm + p) : p;
    Qp[v] = scale_to_half8(__ldg(Q + src * vec_per_node + c), f16_scale_from_n2max(stat[c / vec_per_head].q_n2max));
}

}  // namespace

// After launch_plan (offsets validated) and, when the rows are reordered, after launch_reorder_queries.
cudaError_t launch_f16_convert(const FwdArgs& a, const FwdWorkspace& w) {
    const StatusBlock* sb = reinterpret_cast<const StatusBlock*>(a.ws);
    F16HeadStat* stat = reinterpret_cast<F16HeadStat*>(a.ws + w.f16stat_off);
    cudaError_t err = cudaMemsetAsync(stat, 0, sizeof(F16HeadStat) * (size_t)a.H, a.stream);
    if (err != cudaSuccess) return err;
    const long long n_rows = (long long)a.N * a.H;
    const unsigned row_blocks = (unsigned)((n_rows + 255) / 256);
    const __nv_bfloat16* Q = static_cast<const __nv_bfloat16*>(a.Q);
    const __nv_bfloat16* K = static_cast<const __nv_bfloat16*>(a.K);
    if (a.d == 16) f16_norm_max_kernel<16><<<row_blocks, 256, 0, a.stream>>>(Q, K, n_rows, a.H, reinterpret_cast<unsigned*>(stat), sb);
    else f16_norm_max_kernel<32><<<row_blocks, 256, 0, a.stream>>>(Q, K, n_rows, a.H, reinterpret_cast<unsigned*>(stat), sb);
    const int vec_per_head = a.d * 2 / 16;
    const long long n_vec = n_rows * vec_per_head;
    const unsigned vec_blocks = (unsigned)((n_vec + 255) / 256);
    f16_convert_keys_kernel<<<vec_blocks, 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.K), reinterpret_cast<uint4*>(a.ws + w.kpack_off), n_vec, (int)a.N, a.H, vec_per_head, stat, sb);
    f16_convert_queries_kernel<<<vec_blocks, 256, 0, a.stream>>>(
        static_cast<const uint4*>(a.Q), w.reorder ? reinterpret_cast<const int*>(a.ws + w.perm_off) : nullptr,
        reinterpret_cast<uint4*>(a.ws + w.qperm_off), n_vec, a.H * vec_per_head, vec_per_head, stat, sb);
    return cudaGetLastError();
}

}  // namespace kmip
