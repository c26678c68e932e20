// The full multi-head k-MIP self-attention layer of Eq. 2 (Algorithm 1 with its "Require" line and
// line 8), bf16: Q^h = X W_Q^h, K^h = X W_K^h, V^h = X W_V^h, O^h = kMIP-Attn(Q^h, K^h, V^h) inside each
// graph, Y = sum_h O^h W_O^h, and its backward pass with the selection held constant (Sec. 3.1).
//
// Every dense product runs in gemm_tn.cu (C = A B^T with both operands K-major), so operands are
// brought into that form by two small helpers: padded copies of the weights (a head width that the
// attention kernels do not take - the paper's own study uses d_K = 10 - is zero-padded to 16, 32, 64
// or 128 through zero ROWS of W_Q, W_K, W_V and zero COLUMNS of W_O, which leaves every inner product
// unchanged; the softmax still divides by sqrt(d_head) because the Q projection is scaled by
// sqrt(d_pad / d_head)), and transposes of the activations for the weight gradients.
//   forward   [Q | K | V] = X [W_Q; W_K; W_V]^T   one launch, three output layers, X read once
//             attention core (kmip_attn_forward)
//             Y = O W_O^T
//   backward  dO = dY W_O;  attention backward (dQ, dK, dV);
//             dX = dQ W_Q + dK W_K + dV W_V       one launch, three K segments
//             dW_Q = dQ^T X, dW_K = dK^T X, dW_V = dV^T X   one launch, three output layers, X^T read once
//             dW_O = dY^T O
#include "common.cuh"

namespace kmip {

namespace {

// dst[r, c] = scale * src[map(r), c] for r < rows_pad: rows with r % pad >= real are zero (head padding of W_Q, W_K, W_V)
__global__ void pad_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows_pad, int cols,
                                int pad, int real, float scale) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)rows_pad * cols) return;
    const int r = (int)(i / cols), c = (int)(i % cols), rr = r % pad;
    dst[i] = rr < real ? __float2bfloat16_rn(__bfloat162float(src[(size_t)((r / pad) * real + rr) * cols + c]) * scale)
                       : __float2bfloat16_rn(0.0f);
}
// dst[r, c] = src[r, map(c)] for c < cols_pad: columns with c % pad >= real are zero (head padding of W_O)
__global__ void pad_cols_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int cols_pad,
                                int pad, int real) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)rows * cols_pad) return;
    const int r = (int)(i / cols_pad), c = (int)(i % cols_pad), cc = c % pad;
    const int cols = cols_pad / pad * real;
    dst[i] = cc < real ? src[(size_t)r * cols + (c / pad) * real + cc] : __float2bfloat16_rn(0.0f);
}

// dst[c, r] = src[r, c] for a bf16 matrix [rows, cols]; ld_dst elements between rows of dst (>= rows, a multiple of 8,
// the tail of a row is left untouched and never read: TMA clips at `rows`)
__global__ void transpose_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int cols,
                                 long long ld_dst) {
    __shared__ __nv_bfloat16 tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int y = threadIdx.y; y < 32; y += blockDim.y) {
        const int r = r0 + y, c = c0 + threadIdx.x;
        if (r < rows && c < cols) tile[y][threadIdx.x] = src[(size_t)r * cols + c];
    }
    __syncthreads();
    for (int y = threadIdx.y; y < 32; y += blockDim.y) {
        const int c = c0 + y, r = r0 + threadIdx.x;
        if (r < rows && c < cols) dst[(size_t)c * ld_dst + r] = tile[threadIdx.x][y];
    }
}

// A device-side problem of the attention call (its own status block) becomes the layer call's status.
__global__ void merge_status_kernel(StatusBlock* __restrict__ layer, const StatusBlock* __restrict__ attn) {
    if (attn->status != KMIP_OK) record_status(layer, attn->status, attn->detail);
}

cudaError_t transpose(const void* src, void* dst, int rows, int cols, long long ld_dst, cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    const dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
    transpose_kernel<<<grid, block, 0, stream>>>(static_cast<const __nv_bfloat16*>(src), static_cast<__nv_bfloat16*>(dst), rows,
                                                 cols, ld_dst);
    return cudaGetLastError();
}

}  // namespace

int layer_pad_width(int d_head) { return d_head <= 16 ? 16 : d_head <= 32 ? 32 : d_head <= 64 ? 64 : 128; }

LayerWorkspace plan_layer_workspace(int64_t N, int32_t G, int32_t d_model, int32_t H, int32_t d_head, int32_t k, int pass) {
    LayerWorkspace w;
    const int d_pad = layer_pad_width(d_head);
    const size_t hp = (size_t)H * d_pad, wbytes = hp * d_model * 2;
    const size_t ldn = (size_t)((N + 7) / 8 * 8);  // row pitch of the transposed activations
    size_t o = kStatusBytes;
    auto take = [&o](size_t bytes) { const size_t at = o; o = align_up(o + bytes); return at; };
    w.wq_pad = take(wbytes); w.wk_pad = take(wbytes); w.wv_pad = take(wbytes); w.wo_pad = take(wbytes);
    if (pass == KMIP_PASS_FORWARD) {
        w.attn = take(0);
        w.attn_bytes = plan_fwd_workspace(N, G > 0 ? G : 1, H, d_pad, k, KMIP_BF16_TC).total;
        o = align_up(o + w.attn_bytes);
    } else {
        // transposed padded weights [d_model, H*d_pad] x 3 and [H*d_pad, d_model] of W_O; dO, dQ, dK, dV [N, H*d_pad];
        // transposes of X, dY [d_model, N], of O, dQ, dK, dV [H*d_pad, N]
        w.wqT = take(wbytes); w.wkT = take(wbytes); w.wvT = take(wbytes); w.woT = take(wbytes);
        w.d_o = take((size_t)N * hp * 2); w.d_q = take((size_t)N * hp * 2); w.d_k = take((size_t)N * hp * 2);
        w.d_v = take((size_t)N * hp * 2);
        w.xT = take((size_t)d_model * ldn * 2); w.dyT = take((size_t)d_model * ldn * 2);
        w.oT = take(hp * ldn * 2); w.dqT = take(hp * ldn * 2); w.dkT = take(hp * ldn * 2); w.dvT = take(hp * ldn * 2);
        w.attn = take(0);
        w.attn_bytes = plan_bwd_workspace(N, H, k).total;
        o = align_up(o + w.attn_bytes);
    }
    w.total = o;
    return w;
}

// Padded weight copies shared by both passes: W_Q (scaled), W_K, W_V with zero rows, W_O with zero columns.
static cudaError_t pad_weights(const LayerArgs& a, const LayerWorkspace& w, int d_pad, float q_scale) {
    const int hp = a.H * d_pad;
    const long long n = (long long)hp * a.d_model;
    const unsigned blocks = (unsigned)((n + 255) / 256);
    auto P = [&](size_t off) { return reinterpret_cast<__nv_bfloat16*>(a.ws + off); };
    auto S = [](const void* p) { return static_cast<const __nv_bfloat16*>(p); };
    pad_rows_kernel<<<blocks, 256, 0, a.stream>>>(S(a.w_q), P(w.wq_pad), hp, a.d_model, d_pad, a.d_head, q_scale);
    pad_rows_kernel<<<blocks, 256, 0, a.stream>>>(S(a.w_k), P(w.wk_pad), hp, a.d_model, d_pad, a.d_head, 1.0f);
    pad_rows_kernel<<<blocks, 256, 0, a.stream>>>(S(a.w_v), P(w.wv_pad), hp, a.d_model, d_pad, a.d_head, 1.0f);
    pad_cols_kernel<<<blocks, 256, 0, a.stream>>>(S(a.w_o), P(w.wo_pad), a.d_model, hp, d_pad, a.d_head);
    return cudaGetLastError();
}

// Returns a kmip_status_t.
int layer_forward(const LayerArgs& a) {
    const int d_pad = layer_pad_width(a.d_head), hp = a.H * d_pad;
    const LayerWorkspace w = plan_layer_workspace(a.N, a.G, a.d_model, a.H, a.d_head, a.k, KMIP_PASS_FORWARD);
    StatusBlock* sb = reinterpret_cast<StatusBlock*>(a.ws);
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    // the Q projection carries sqrt(d_pad / d_head): the core divides by sqrt(d_pad), Eq. 1 by sqrt(d_head)
    if (pad_weights(a, w, d_pad, sqrtf((float)d_pad / (float)a.d_head)) != cudaSuccess) return KMIP_ERR_CUDA;
    const void* A[3] = {a.x, a.x, a.x};
    const void* B[3] = {a.ws + w.wq_pad, a.ws + w.wk_pad, a.ws + w.wv_pad};
    void* C[3] = {a.q, a.k_proj, a.v};
    if (launch_gemm_tn(A, a.d_model, B, a.d_model, C, nullptr, 3, 1, (int)a.N, hp, a.d_model, hp, 0, 0, 0, 0, false, sb,
                       a.stream) != cudaSuccess)
        return KMIP_ERR_CUDA;
    const int rc = kmip_attn_forward(a.q, a.k_proj, a.v, a.graph_offsets, a.G, a.N, a.H, d_pad, a.k, KMIP_BF16_TC, a.o,
                                     a.topk_idx, a.topk_score, a.ws + w.attn, w.attn_bytes, a.stream);
    if (rc != KMIP_OK) return rc;
    merge_status_kernel<<<1, 1, 0, a.stream>>>(sb, reinterpret_cast<const StatusBlock*>(a.ws + w.attn));
    const void* A2[3] = {a.o, a.o, a.o};
    const void* B2[3] = {a.ws + w.wo_pad, a.ws + w.wo_pad, a.ws + w.wo_pad};
    void* C2[3] = {a.y, a.y, a.y};
    if (launch_gemm_tn(A2, hp, B2, hp, C2, nullptr, 1, 1, (int)a.N, a.d_model, hp, a.d_model, 0, 0, 0, 0, false, sb, a.stream) !=
        cudaSuccess)
        return KMIP_ERR_CUDA;
    return KMIP_OK;
}

int layer_backward(const LayerArgs& a) {
    const int d_pad = layer_pad_width(a.d_head), hp = a.H * d_pad, N = (int)a.N;
    const LayerWorkspace w = plan_layer_workspace(a.N, a.G, a.d_model, a.H, a.d_head, a.k, KMIP_PASS_BACKWARD);
    StatusBlock* sb = reinterpret_cast<StatusBlock*>(a.ws);
    const long long ldn = (a.N + 7) / 8 * 8;
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    const float q_scale = sqrtf((float)d_pad / (float)a.d_head);
    if (pad_weights(a, w, d_pad, q_scale) != cudaSuccess) return KMIP_ERR_CUDA;
    auto P = [&](size_t off) { return static_cast<void*>(a.ws + off); };
    // transposes of the padded weights: W^T [d_model, H*d_pad] for dX, W_O^T [H*d_pad, d_model] for dO
    if (transpose(P(w.wq_pad), P(w.wqT), hp, a.d_model, hp, a.stream) != cudaSuccess ||
        transpose(P(w.wk_pad), P(w.wkT), hp, a.d_model, hp, a.stream) != cudaSuccess ||
        transpose(P(w.wv_pad), P(w.wvT), hp, a.d_model, hp, a.stream) != cudaSuccess ||
        transpose(P(w.wo_pad), P(w.woT), a.d_model, hp, a.d_model, a.stream) != cudaSuccess)
        return KMIP_ERR_CUDA;
    // dO = dY W_O (padded columns come out zero)
    {
        const void* A[3] = {a.d_y, a.d_y, a.d_y};
        const void* B[3] = {P(w.woT), P(w.woT), P(w.woT)};
        void* C[3] = {P(w.d_o), P(w.d_o), P(w.d_o)};
        if (launch_gemm_tn(A, a.d_model, B, a.d_model, C, nullptr, 1, 1, N, hp, a.d_model, hp, 0, 0, 0, 0, false, sb, a.stream) !=
            cudaSuccess)
            return KMIP_ERR_CUDA;
    }
    const int rc = kmip_attn_backward(a.q, a.k_proj, a.v, a.graph_offsets, a.G, a.N, a.H, d_pad, a.k, KMIP_BF16_TC, a.o, P(w.d_o),
                                      a.topk_idx, a.topk_score, P(w.d_q), P(w.d_k), P(w.d_v), a.ws + w.attn, w.attn_bytes,
                                      a.stream);
    if (rc != KMIP_OK) return rc;
    merge_status_kernel<<<1, 1, 0, a.stream>>>(sb, reinterpret_cast<const StatusBlock*>(a.ws + w.attn));
    // dX = dQ' W_Q' + dK W_K + dV W_V with the scaled, padded W_Q' (its scale is the chain rule of Q' = s Q)
    {
        const void* A[3] = {P(w.d_q), P(w.d_k), P(w.d_v)};
        const void* B[3] = {P(w.wqT), P(w.wkT), P(w.wvT)};
        void* C[3] = {a.d_x, a.d_x, a.d_x};
        if (launch_gemm_tn(A, hp, B, hp, C, nullptr, 1, 3, N, a.d_model, hp, a.d_model, 0, 0, 0, 0, false, sb, a.stream) !=
            cudaSuccess)
            return KMIP_ERR_CUDA;
    }
    // weight gradients: the node axis becomes the contraction
    if (transpose(a.x, P(w.xT), N, a.d_model, ldn, a.stream) != cudaSuccess ||
        transpose(a.d_y, P(w.dyT), N, a.d_model, ldn, a.stream) != cudaSuccess ||
        transpose(a.o, P(w.oT), N, hp, ldn, a.stream) != cudaSuccess ||
        transpose(P(w.d_q), P(w.dqT), N, hp, ldn, a.stream) != cudaSuccess ||
        transpose(P(w.d_k), P(w.dkT), N, hp, ldn, a.stream) != cudaSuccess ||
        transpose(P(w.d_v), P(w.dvT), N, hp, ldn, a.stream) != cudaSuccess)
        return KMIP_ERR_CUDA;
    {
        // dW_Q = s dQ'^T X (rows of the padding dropped), dW_K, dW_V alike: X^T shared by the three layers
        const void* A[3] = {P(w.dqT), P(w.dkT), P(w.dvT)};
        const void* B[3] = {P(w.xT), P(w.xT), P(w.xT)};
        void* C[3] = {a.dw_q, a.dw_k, a.dw_v};
        const float sc[3] = {q_scale, 1.0f, 1.0f};
        // batched over A here: the kernel batches over B, so the roles are swapped through C^T = B A^T ... instead
        // three launches keep the code plain (the weights are small)
        for (int z = 0; z < 3; ++z) {
            const void* Az[3] = {A[z], A[z], A[z]};
            void* Cz[3] = {C[z], C[z], C[z]};
            const float sz[3] = {sc[z], sc[z], sc[z]};
            if (launch_gemm_tn(Az, (int)ldn, B, (int)ldn, Cz, sz, 1, 1, hp, a.d_model, N, a.d_model, d_pad, a.d_head, 0, 0, false,
                               sb, a.stream) != cudaSuccess)
                return KMIP_ERR_CUDA;
        }
    }
    {
        // dW_O = dY^T O (columns of the padding dropped)
        const void* A[3] = {P(w.dyT), P(w.dyT), P(w.dyT)};
        const void* B[3] = {P(w.oT), P(w.oT), P(w.oT)};
        void* C[3] = {a.dw_o, a.dw_o, a.dw_o};
        if (launch_gemm_tn(A, (int)ldn, B, (int)ldn, C, nullptr, 1, 1, a.d_model, hp, N, a.H * a.d_head, 0, 0, d_pad, a.d_head,
                           false, sb, a.stream) != cudaSuccess)
            return KMIP_ERR_CUDA;
    }
    return KMIP_OK;
}

}  // namespace kmip
