// C ABI of the k-MIP attention library: argument validation and kernel sequencing.
// Nothing here allocates device memory or synchronises the stream (kmip_last_status excepted).
#include "common.cuh"
#include "kmip_test.h"

using namespace kmip;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int64_t N, int32_t H, int32_t d, int32_t k, int mode) {
    if (N < 0 || N >= (int64_t)1 << 31 || H < 1 || k < 1 || d < 1) return KMIP_ERR_INVALID_ARG;
    if (mode != KMIP_BF16_TC && mode != KMIP_FP32_EXACT && mode != KMIP_BF16_TC_PRUNED) return KMIP_ERR_UNSUPPORTED;
    if (d != 16 && d != 32 && d != 64 && d != 128) return KMIP_ERR_UNSUPPORTED;
    if (k > 128) return KMIP_ERR_UNSUPPORTED;
    if ((__int128)N * H * k >= (__int128)1 << 31) return KMIP_ERR_INVALID_ARG;
    if ((__int128)N * H * d >= (__int128)1 << 40) return KMIP_ERR_INVALID_ARG;
    return KMIP_OK;
}

// ---- optional per-stage timing (off unless kmip_profile_enable was called) ----------------------
constexpr int kProfMaxCalls = 256;
struct Profile {
    bool on = false;
    int max_calls = 0;
    int n_fwd = 0, n_bwd = 0;
    cudaEvent_t fwd[kProfMaxCalls][5];
    cudaEvent_t bwd[kProfMaxCalls][4];
};
Profile g_prof;

int forward_impl(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G, int64_t N,
                 int32_t H, int32_t d, int32_t k, int mode, float drop_p, uint64_t seed, void* out,
                 int32_t* topk_idx, float* topk_score, void* workspace, size_t workspace_bytes, void* stream,
                 const kmip_test_options_t* opt);

}  // namespace

extern "C" {

int kmip_version(void) { return 200; }

int kmip_build_flags(void) { return kChecks ? 1 : 0; }

const char* kmip_status_string(int status) {
    switch (status) {
        case KMIP_OK: return "ok";
        case KMIP_ERR_INVALID_ARG: return "invalid argument";
        case KMIP_ERR_UNSUPPORTED: return "unsupported head width, k or mode";
        case KMIP_ERR_WORKSPACE: return "workspace too small";
        case KMIP_ERR_CUDA: return "CUDA runtime or launch failure";
        case KMIP_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case KMIP_ERR_BAD_OFFSETS: return "graph_offsets is not a valid CSR offset array";
        case KMIP_ERR_TOO_LARGE: return "problem needs more scratch than the library's built-in array holds";
        case KMIP_ERR_CHECK: return "a device-side index test or workspace canary of a KMIP_CHECKS build failed";
        default: return "unknown status";
    }
}

int kmip_attn_workspace_bytes(int64_t N, int32_t G, int32_t H, int32_t d, int32_t k, int mode, int pass,
                              size_t* bytes) {
    if (!bytes || G < 0) return KMIP_ERR_INVALID_ARG;
    const int rc = check_shape(N, H, d, k, mode);
    if (rc != KMIP_OK) return rc;
    if (pass == KMIP_PASS_FORWARD)
        *bytes = plan_fwd_workspace(N, G, H, d, k, mode).total;
    else if (pass == KMIP_PASS_BACKWARD) *bytes = plan_bwd_workspace(N, H, k).total;
    else return KMIP_ERR_INVALID_ARG;
    return KMIP_OK;
}

int kmip_attn_forward(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G,
                      int64_t N, int32_t H, int32_t d, int32_t k, int mode, void* out, int32_t* topk_idx,
                      float* topk_score, void* workspace, size_t workspace_bytes, void* stream) {
    return kmip_attn_forward_dropout(Q, K, V, graph_offsets, G, N, H, d, k, mode, 0.0f, 0ull, out, topk_idx, topk_score,
                                     workspace, workspace_bytes, stream);
}

int kmip_attn_forward_dropout(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G,
                              int64_t N, int32_t H, int32_t d, int32_t k, int mode, float drop_p, uint64_t seed,
                              void* out, int32_t* topk_idx, float* topk_score, void* workspace,
                              size_t workspace_bytes, void* stream) {
    return forward_impl(Q, K, V, graph_offsets, G, N, H, d, k, mode, drop_p, seed, out, topk_idx, topk_score, workspace,
                        workspace_bytes, stream, nullptr);
}

int kmip_test_attn_forward(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G,
                           int64_t N, int32_t H, int32_t d, int32_t k, int mode, void* out, int32_t* topk_idx,
                           float* topk_score, void* workspace, size_t workspace_bytes, void* stream,
                           const kmip_test_options_t* options) {
    return forward_impl(Q, K, V, graph_offsets, G, N, H, d, k, mode, 0.0f, 0ull, out, topk_idx, topk_score, workspace,
                        workspace_bytes, stream, options);
}

}  // extern "C"

namespace {

int forward_impl(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G, int64_t N,
                 int32_t H, int32_t d, int32_t k, int mode, float drop_p, uint64_t seed, void* out,
                 int32_t* topk_idx, float* topk_score, void* workspace, size_t workspace_bytes, void* stream,
                 const kmip_test_options_t* opt) {
    const int rc = check_shape(N, H, d, k, mode);
    if (rc != KMIP_OK) return rc;
    if (!(drop_p >= 0.0f && drop_p < 1.0f)) return KMIP_ERR_INVALID_ARG;
    if (N == 0) return KMIP_OK;
    if (graph_offsets != nullptr && G < 1) return KMIP_ERR_INVALID_ARG;
    if (!Q || !K || !V || !out || !topk_idx || !topk_score || !workspace) return KMIP_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out) || !aligned16(topk_idx) ||
        !aligned16(topk_score) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(graph_offsets) & 3u))
        return KMIP_ERR_INVALID_ARG;
    const FwdWorkspace w = plan_fwd_workspace(N, graph_offsets ? G : 1, H, d, k, mode);
    const bool tc = w.tc;
    if (workspace_bytes < w.total) return KMIP_ERR_WORKSPACE;

    FwdArgs a{Q, K, V, graph_offsets, graph_offsets ? G : 1, N, H, d, k, mode, out, topk_idx, topk_score,
              static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)};
    a.drop_p = drop_p;
    a.seed = seed;
    if (opt) {
        a.wait_limit_cycles = opt->wait_limit_cycles;
        a.drop_first_tile = opt->drop_first_tile;
        a.fp32_path = opt->fp32_path;
    }
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_canary_fill(a.ws, w.canaries, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    cudaEvent_t* ev = (g_prof.on && g_prof.n_fwd < g_prof.max_calls) ? g_prof.fwd[g_prof.n_fwd++] : nullptr;
    if (ev) cudaEventRecord(ev[0], a.stream);
    if (tc && !w.prune && !w.f16 && launch_pack_keys(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    // the tiled fp32 sweep runs one block per 128 query rows and head and reads a key once per block instead of
    // once per row: measured faster than the one-warp-per-row kernel from about 48 blocks on (0.43 against
    // 0.70 ms at 64 blocks, 1.7 against 8.4 ms at 247), slower below (0.25 against 0.19 ms at 32)
    const bool tiled32 = mode == KMIP_FP32_EXACT && score_select_fp32_tiled_supported(d, k) &&
                         (a.fp32_path == 0 ? (N / 128) * H >= 48 : a.fp32_path == 2);
    if (launch_plan(a, w, w.f16 ? score_select_f16_rows_per_item(k) : tc ? score_select_tc_rows_per_item(d, k) : 128) !=
        cudaSuccess)
        return KMIP_ERR_CUDA;
    if (w.reorder && launch_reorder_queries(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    if (w.f16 && launch_f16_convert(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    if (w.prune && (launch_reorder_keys(a, w) != cudaSuccess || launch_prune_stats(a, w) != cudaSuccess)) return KMIP_ERR_CUDA;
    if (ev) cudaEventRecord(ev[1], a.stream);
    const cudaError_t sweep = w.f16 ? launch_score_select_f16(a, w) : tc ? launch_score_select_tc(a, w)
                              : tiled32 ? launch_score_select_fp32_tiled(a, w) : launch_score_select_exact(a);
    if (sweep != cudaSuccess) return KMIP_ERR_CUDA;
    if (ev) cudaEventRecord(ev[2], a.stream);
    if (w.f16 && (launch_refine_f16(a, w) != cudaSuccess || launch_score_select_exact_redo(a, w) != cudaSuccess))
        return KMIP_ERR_CUDA;
    if (tc && !w.f16 && launch_refine_topk(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    if (tiled32 && launch_refine_topk_fp32(a) != cudaSuccess) return KMIP_ERR_CUDA;
    if (ev) cudaEventRecord(ev[3], a.stream);
    if (launch_softmax_gather(a) != cudaSuccess) return KMIP_ERR_CUDA;
    if (ev) cudaEventRecord(ev[4], a.stream);
    if (launch_canary_check(a.ws, w.canaries, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    return KMIP_OK;
}

}  // namespace

extern "C" {

int kmip_attn_backward(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G,
                       int64_t N, int32_t H, int32_t d, int32_t k, int mode, const void* out, const void* d_out,
                       const int32_t* topk_idx, const float* topk_score, void* dQ, void* dK, void* dV,
                       void* workspace, size_t workspace_bytes, void* stream) {
    return kmip_attn_backward_dropout(Q, K, V, graph_offsets, G, N, H, d, k, mode, 0.0f, 0ull, out, d_out, topk_idx,
                                      topk_score, dQ, dK, dV, workspace, workspace_bytes, stream);
}

int kmip_attn_backward_dropout(const void* Q, const void* K, const void* V, const int32_t* graph_offsets, int32_t G,
                               int64_t N, int32_t H, int32_t d, int32_t k, int mode, float drop_p, uint64_t seed,
                               const void* out, const void* d_out, const int32_t* topk_idx, const float* topk_score,
                               void* dQ, void* dK, void* dV, void* workspace, size_t workspace_bytes, void* stream) {
    (void)graph_offsets; (void)G; (void)out;
    const int rc = check_shape(N, H, d, k, mode);
    if (rc != KMIP_OK) return rc;
    if (!(drop_p >= 0.0f && drop_p < 1.0f)) return KMIP_ERR_INVALID_ARG;
    if (N == 0) return KMIP_OK;
    if (!Q || !K || !V || !d_out || !topk_idx || !topk_score || !dQ || !dK || !dV || !workspace)
        return KMIP_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(d_out) || !aligned16(topk_idx) ||
        !aligned16(topk_score) || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(workspace))
        return KMIP_ERR_INVALID_ARG;
    const BwdWorkspace w = plan_bwd_workspace(N, H, k);
    if (workspace_bytes < w.total) return KMIP_ERR_WORKSPACE;
    BwdArgs a{Q, K, V, d_out, N, H, d, k, mode, topk_idx, topk_score, dQ, dK, dV,
              static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)};
    a.drop_p = drop_p;
    a.seed = seed;
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_canary_fill(a.ws, w.canaries, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    cudaEvent_t* ev = (g_prof.on && g_prof.n_bwd < g_prof.max_calls) ? g_prof.bwd[g_prof.n_bwd++] : nullptr;
    if (ev) cudaEventRecord(ev[0], a.stream);
    if (launch_backward(a, w, ev ? ev + 1 : nullptr) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_canary_check(a.ws, w.canaries, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    return KMIP_OK;
}

int kmip_attn_topk_mass(const void* Q, const void* K, const int32_t* graph_offsets, int32_t G, int64_t N, int32_t H,
                        int32_t d, int32_t k, int mode, const float* topk_score, float* mass, void* workspace,
                        size_t workspace_bytes, void* stream) {
    const int rc = check_shape(N, H, d, k, mode);
    if (rc != KMIP_OK) return rc;
    const bool tensor = mode != KMIP_FP32_EXACT;  // bf16 storage: the scores come from the tensor cores
    if (!tensor && d > 64) return KMIP_ERR_UNSUPPORTED;
    if (N == 0) return KMIP_OK;
    if (graph_offsets != nullptr && G < 1) return KMIP_ERR_INVALID_ARG;
    if (!Q || !K || !topk_score || !mass || !workspace) return KMIP_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(topk_score) || !aligned16(workspace) ||
        (reinterpret_cast<uintptr_t>(mass) & 3u) || (reinterpret_cast<uintptr_t>(graph_offsets) & 3u))
        return KMIP_ERR_INVALID_ARG;
    const FwdWorkspace w = plan_fwd_workspace(N, graph_offsets ? G : 1, H, d, k, mode,
                                              tensor ? kPlanTcFp32AccInOrder : kPlanNoTensorCore);
    if (workspace_bytes < w.total) return KMIP_ERR_WORKSPACE;
    FwdArgs a{Q, K, nullptr, graph_offsets, graph_offsets ? G : 1, N, H, d, k, mode, nullptr, nullptr,
              const_cast<float*>(topk_score), static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)};
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    if (tensor) {
        if (launch_pack_keys(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
        if (launch_plan(a, w, score_select_tc_rows_per_item(d, 1)) != cudaSuccess) return KMIP_ERR_CUDA;
        if (launch_topk_mass_tc(a, w, mass) != cudaSuccess) return KMIP_ERR_CUDA;
        return KMIP_OK;
    }
    if (launch_plan(a, w, 128) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_topk_mass(a, w, mass) != cudaSuccess) return KMIP_ERR_CUDA;
    return KMIP_OK;
}

static int check_layer(const kmip_layer_tensors_t* t, int64_t N, int32_t G, int32_t d_model, int32_t H, int32_t d_head, int32_t k,
                       bool backward) {
    if (d_head < 1 || d_head > 128 || d_model < 8 || (d_model & 7) || G < 0) return d_head > 128 ? KMIP_ERR_UNSUPPORTED : KMIP_ERR_INVALID_ARG;
    const int rc = check_shape(N, H, layer_pad_width(d_head), k, KMIP_BF16_TC);
    if (rc != KMIP_OK) return rc;
    if (!t) return KMIP_ERR_INVALID_ARG;
    const void* need_f[] = {t->x, t->w_q, t->w_k, t->w_v, t->w_o, t->q, t->k, t->v, t->o, t->topk_idx, t->topk_score};
    for (const void* p : need_f)
        if (!p || !aligned16(p)) return KMIP_ERR_INVALID_ARG;
    if (!backward && (!t->y || !aligned16(t->y))) return KMIP_ERR_INVALID_ARG;
    if (backward) {
        const void* need_b[] = {t->d_y, t->d_x, t->dw_q, t->dw_k, t->dw_v, t->dw_o};
        for (const void* p : need_b)
            if (!p || !aligned16(p)) return KMIP_ERR_INVALID_ARG;
    }
    return KMIP_OK;
}

static LayerArgs layer_args(const kmip_layer_tensors_t* t, const int32_t* graph_offsets, int32_t G, int64_t N, int32_t d_model,
                            int32_t H, int32_t d_head, int32_t k, void* workspace, void* stream) {
    LayerArgs a{};
    a.x = t->x; a.w_q = t->w_q; a.w_k = t->w_k; a.w_v = t->w_v; a.w_o = t->w_o;
    a.q = t->q; a.k_proj = t->k; a.v = t->v; a.o = t->o;
    a.topk_idx = t->topk_idx; a.topk_score = t->topk_score;
    a.y = t->y; a.d_y = t->d_y;
    a.d_x = t->d_x; a.dw_q = t->dw_q; a.dw_k = t->dw_k; a.dw_v = t->dw_v; a.dw_o = t->dw_o;
    a.graph_offsets = graph_offsets; a.G = graph_offsets ? G : 1; a.N = N;
    a.d_model = d_model; a.H = H; a.d_head = d_head; a.k = k;
    a.ws = static_cast<unsigned char*>(workspace);
    a.stream = static_cast<cudaStream_t>(stream);
    return a;
}

int kmip_layer_workspace_bytes(int64_t N, int32_t G, int32_t d_model, int32_t H, int32_t d_head, int32_t k, int pass,
                               size_t* bytes) {
    if (!bytes || (pass != KMIP_PASS_FORWARD && pass != KMIP_PASS_BACKWARD)) return KMIP_ERR_INVALID_ARG;
    if (d_head < 1 || d_model < 8 || (d_model & 7) || G < 0) return KMIP_ERR_INVALID_ARG;
    if (d_head > 128) return KMIP_ERR_UNSUPPORTED;
    const int rc = check_shape(N, H, layer_pad_width(d_head), k, KMIP_BF16_TC);
    if (rc != KMIP_OK) return rc;
    *bytes = plan_layer_workspace(N, G, d_model, H, d_head, k, pass).total;
    return KMIP_OK;
}

int kmip_layer_forward(const kmip_layer_tensors_t* t, const int32_t* graph_offsets, int32_t G, int64_t N, int32_t d_model,
                       int32_t H, int32_t d_head, int32_t k, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_layer(t, N, G, d_model, H, d_head, k, false);
    if (rc != KMIP_OK) return rc;
    if (N == 0) return KMIP_OK;
    if ((graph_offsets != nullptr && G < 1) || !workspace || !aligned16(workspace)) return KMIP_ERR_INVALID_ARG;
    if (workspace_bytes < plan_layer_workspace(N, graph_offsets ? G : 1, d_model, H, d_head, k, KMIP_PASS_FORWARD).total)
        return KMIP_ERR_WORKSPACE;
    return layer_forward(layer_args(t, graph_offsets, G, N, d_model, H, d_head, k, workspace, stream));
}

int kmip_layer_backward(const kmip_layer_tensors_t* t, const int32_t* graph_offsets, int32_t G, int64_t N, int32_t d_model,
                        int32_t H, int32_t d_head, int32_t k, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_layer(t, N, G, d_model, H, d_head, k, true);
    if (rc != KMIP_OK) return rc;
    if (N == 0) return KMIP_OK;
    if ((graph_offsets != nullptr && G < 1) || !workspace || !aligned16(workspace)) return KMIP_ERR_INVALID_ARG;
    if (workspace_bytes < plan_layer_workspace(N, graph_offsets ? G : 1, d_model, H, d_head, k, KMIP_PASS_BACKWARD).total)
        return KMIP_ERR_WORKSPACE;
    return layer_backward(layer_args(t, graph_offsets, G, N, d_model, H, d_head, k, workspace, stream));
}

int kmip_last_status(const void* workspace, void* stream, int* device_status) {
    if (!workspace || !device_status) return KMIP_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return KMIP_ERR_CUDA;
    int st = 0;
    if (cudaMemcpy(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return KMIP_ERR_CUDA;
    *device_status = st;
    return KMIP_OK;
}

int kmip_attn_sweep_counters(const void* workspace, void* stream, int64_t* counters) {
    if (!workspace || !counters) return KMIP_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return KMIP_ERR_CUDA;
    StatusBlock sb;
    if (cudaMemcpy(&sb, workspace, sizeof(sb), cudaMemcpyDeviceToHost) != cudaSuccess) return KMIP_ERR_CUDA;
    for (int i = 0; i < 4; ++i) counters[i] = (int64_t)sb.counters[i];
    counters[4] = sb.n_redo;
    counters[5] = counters[6] = counters[7] = 0;
    return KMIP_OK;
}

int kmip_profile_enable(int max_calls) {
    if (g_prof.on) {
        for (int i = 0; i < g_prof.max_calls; ++i) {
            for (int e = 0; e < 5; ++e) cudaEventDestroy(g_prof.fwd[i][e]);
            for (int e = 0; e < 4; ++e) cudaEventDestroy(g_prof.bwd[i][e]);
        }
        g_prof.on = false;
    }
    g_prof.n_fwd = g_prof.n_bwd = 0;
    g_prof.max_calls = 0;
    if (max_calls <= 0) return KMIP_OK;
    if (max_calls > kProfMaxCalls) max_calls = kProfMaxCalls;
    for (int i = 0; i < max_calls; ++i) {
        for (int e = 0; e < 5; ++e)
            if (cudaEventCreate(&g_prof.fwd[i][e]) != cudaSuccess) return KMIP_ERR_CUDA;
        for (int e = 0; e < 4; ++e)
            if (cudaEventCreate(&g_prof.bwd[i][e]) != cudaSuccess) return KMIP_ERR_CUDA;
    }
    g_prof.max_calls = max_calls;
    g_prof.on = true;
    return KMIP_OK;
}

int kmip_profile_read(double* stage_ms, int* calls) {
    if (!stage_ms || !calls) return KMIP_ERR_INVALID_ARG;
    for (int s = 0; s < 7; ++s) stage_ms[s] = 0.0;
    calls[0] = g_prof.n_fwd;
    calls[1] = g_prof.n_bwd;
    if (!g_prof.on) return KMIP_OK;
    for (int pass = 0; pass < 2; ++pass) {
        const int n = pass ? g_prof.n_bwd : g_prof.n_fwd;
        const int n_stage = pass ? 3 : 4;
        for (int i = 0; i < n; ++i) {
            cudaEvent_t* ev = pass ? g_prof.bwd[i] : g_prof.fwd[i];
            if (cudaEventSynchronize(ev[n_stage]) != cudaSuccess) return KMIP_ERR_CUDA;
            for (int s = 0; s < n_stage; ++s) {
                float ms = 0.0f;
                if (cudaEventElapsedTime(&ms, ev[s], ev[s + 1]) != cudaSuccess) return KMIP_ERR_CUDA;
                stage_ms[pass * 4 + s] += ms;
            }
        }
    }
    g_prof.n_fwd = g_prof.n_bwd = 0;
    return KMIP_OK;
}

int kmip_test_gemm_tn(const void* A, const void* B, void* C, int32_t M, int32_t N, int32_t K, int out_f32, void* workspace,
                      size_t workspace_bytes, void* stream) {
    if (!A || !B || !C || !workspace || M < 1 || N < 1 || K < 8 || (K & 7)) return KMIP_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C) || !aligned16(workspace)) return KMIP_ERR_INVALID_ARG;
    if (workspace_bytes < kStatusBytes) return KMIP_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, kStatusBytes, st) != cudaSuccess) return KMIP_ERR_CUDA;
    const void* As[3] = {A, A, A};
    const void* Bs[3] = {B, B, B};
    void* Cs[3] = {C, C, C};
    if (launch_gemm_tn(As, K, Bs, K, Cs, nullptr, 1, 1, M, N, K, N, 0, 0, 0, 0, out_f32 != 0, static_cast<StatusBlock*>(workspace),
                       st) != cudaSuccess)
        return KMIP_ERR_CUDA;
    return KMIP_OK;
}

int kmip_test_sweep_order(const void* workspace, int64_t N, int32_t G, int32_t H, int32_t d, int32_t k, int mode,
                          int32_t* order, int32_t* rows_per_item, void* stream) {
    const int rc = check_shape(N, H, d, k, mode);
    if (rc != KMIP_OK) return rc;
    if (!workspace || !order || !rows_per_item || G < 0) return KMIP_ERR_INVALID_ARG;
    const FwdWorkspace w = plan_fwd_workspace(N, G > 0 ? G : 1, H, d, k, mode);
    *rows_per_item = w.f16 ? score_select_f16_rows_per_item(k) : w.tc ? score_select_tc_rows_per_item(d, k) : 128;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return KMIP_ERR_CUDA;
    if (w.reorder) {
        if (cudaMemcpy(order, static_cast<const unsigned char*>(workspace) + w.perm_off, (size_t)N * 4,
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return KMIP_ERR_CUDA;
    } else {
        for (int64_t i = 0; i < N; ++i) order[i] = (int32_t)i;
    }
    return KMIP_OK;
}

// Declared in kmip_test.h: dense scores of the tensor-core pipeline, for element-wise checks of the contraction.
int kmip_test_tc_scores(const void* Q, const void* K, int64_t N, int32_t H, int32_t d, float* scores,
                         void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_shape(N, H, d, 1, KMIP_BF16_TC);
    if (rc != KMIP_OK) return rc;
    if (!Q || !K || !scores || !workspace || N < 1 || N > 8192) return KMIP_ERR_INVALID_ARG;
    const FwdWorkspace w = plan_fwd_workspace(N, 1, H, d, 1, KMIP_BF16_TC, kPlanTcFp32Acc);
    if (workspace_bytes < w.total) return KMIP_ERR_WORKSPACE;
    FwdArgs a{Q, K, nullptr, nullptr, 1, N, H, d, 1, KMIP_BF16_TC, nullptr, nullptr, nullptr,
              static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)};
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_pack_keys(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_plan(a, w, score_select_tc_rows_per_item(d, 1)) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_score_dump_tc(a, w, scores) != cudaSuccess) return KMIP_ERR_CUDA;
    return KMIP_OK;
}

int kmip_test_f16_scores(const void* Q, const void* K, int64_t N, int32_t H, int32_t d, float* scores, float* scales,
                         void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_shape(N, H, d, 1, KMIP_BF16_TC);
    if (rc != KMIP_OK) return rc;
    if (d > 32) return KMIP_ERR_UNSUPPORTED;
    if (!Q || !K || !scores || !scales || !workspace || N < 1 || N > 8192) return KMIP_ERR_INVALID_ARG;
    const FwdWorkspace w = plan_fwd_workspace(N, 1, H, d, 1, KMIP_BF16_TC, kPlanTcFp16Acc);
    if (workspace_bytes < w.total) return KMIP_ERR_WORKSPACE;
    FwdArgs a{Q, K, nullptr, nullptr, 1, N, H, d, 1, KMIP_BF16_TC, nullptr, nullptr, nullptr,
              static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)};
    if (cudaMemsetAsync(a.ws, 0, kStatusBytes, a.stream) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_plan(a, w, score_select_f16_rows_per_item(1)) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_f16_convert(a, w) != cudaSuccess) return KMIP_ERR_CUDA;
    if (launch_score_dump_f16(a, w, scores) != cudaSuccess) return KMIP_ERR_CUDA;
    // per head: {q_n2max, k_n2max, k_first16_n2max, 0} as the conversion measured them
    if (cudaMemcpyAsync(scales, a.ws + w.f16stat_off, sizeof(float) * 4 * (size_t)H, cudaMemcpyDeviceToDevice, a.stream) !=
        cudaSuccess)
        return KMIP_ERR_CUDA;
    return KMIP_OK;
}

}  // extern "C"
