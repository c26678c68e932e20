/*
 * kmip_test.h -- entry points of libkmip.so that exist for its tests, not for applications.
 *
 * They reach code paths that the public calls of kmip.h choose on their own (which fp32 sweep runs)
 * or that only a failure reaches (an expired bounded wait), and expose the raw tensor-core scores
 * so that the contraction of Algorithm 1 line 2 can be checked element by element.  Every option
 * travels with the call: the library keeps no test state, so calls from different host threads
 * cannot influence each other.  The paper has no counterpart for any of them.
 */
#ifndef KMIP_TEST_H_
#define KMIP_TEST_H_

#include "kmip.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    /* Bound of every device-side wait of the tensor-core sweep, in SM clocks; <= 0 keeps the
       library's default (about 4 s).  A wait that runs out sets KMIP_ERR_TIMEOUT in the status
       word and the kernel returns normally. */
    int64_t wait_limit_cycles;
    /* Non-zero: CTA 0 of the tensor-core sweep never loads its first key tile, so the waits on
       that tile must run out (failure detection without a GPU fault). */
    int32_t drop_first_tile;
    /* KMIP_FP32_EXACT only: 0 = the sweep is chosen by problem size, 1 = one warp per query row,
       2 = the tiled sweep whenever it supports (d, k). */
    int32_t fp32_path;
} kmip_test_options_t;

/*
 * kmip_attn_forward (Eq. 1, Algorithm 1 lines 2-6) with per-call test options; `options` may be
 * NULL, which is exactly kmip_attn_forward.  Arguments, layouts, ownership and errors are those
 * of kmip_attn_forward.
 */
int kmip_test_attn_forward(const void *Q, const void *K, const void *V,
                           const int32_t *graph_offsets, int32_t G, int64_t N,
                           int32_t H, int32_t d, int32_t k, int mode,
                           void *out, int32_t *topk_idx, float *topk_score,
                           void *workspace, size_t workspace_bytes, void *stream,
                           const kmip_test_options_t *options);

/*
 * Dense scores S[h][i][j] = q_i^h . k_j^h (Algorithm 1 line 2) of ONE graph of 1 <= N <= 8192 nodes,
 * written as fp32 [H, N, N] to `scores` (device memory) through the same TMA / tcgen05 pipeline as
 * the KMIP_BF16_TC forward pass.  Q, K: bf16 [N, H, d] device memory.  workspace: at least
 * kmip_attn_workspace_bytes(N, 1, H, d, 1, KMIP_BF16_TC, KMIP_PASS_FORWARD) bytes.
 * Errors as for kmip_attn_forward; N outside [1, 8192] is KMIP_ERR_INVALID_ARG.
 */
int kmip_test_tc_scores(const void *Q, const void *K, int64_t N, int32_t H, int32_t d,
                        float *scores, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The scores of the half-precision prefilter sweep (head widths 16 and 32): the tensor-core contraction of
 * the scaled fp16 copies of Q and K with fp16 accumulators, T[h][i][j] ~ s_q[h] s_k[h] (q_i^h . k_j^h), written
 * as fp32 [H, N, N] to `scores` for ONE graph of 1 <= N <= 8192 nodes.  `stats` (device, float [H, 4]) receives
 * per head {largest squared query-row norm, largest squared key-row norm, largest squared norm of the first
 * 16 elements of a key row, 0} as the conversion measured them; the scales s_q, s_k are the powers of two that
 * put the largest norm into [32, 64).  Tests use it to check the error bound the rescoring kernel relies on.
 * workspace: kmip_attn_workspace_bytes(N, 1, H, d, 1, KMIP_BF16_TC, KMIP_PASS_FORWARD) bytes.
 * d > 32 is KMIP_ERR_UNSUPPORTED; other errors as for kmip_test_tc_scores.
 */
int kmip_test_f16_scores(const void *Q, const void *K, int64_t N, int32_t H, int32_t d,
                         float *scores, float *stats, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The dense product behind the layer's projections (Eq. 2) on its own:
 *   C[M, N] = A[M, K] B[N, K]^T,  A and B bf16 row-major device memory with lda = ldb = K (a multiple of 8),
 * C bf16 (out_f32 = 0) or fp32 (out_f32 = 1) row-major with ldc = N, fp32 accumulation on the tensor cores.
 * workspace: at least 256 bytes (status block).  Errors as for kmip_attn_forward.
 */
int kmip_test_gemm_tn(const void *A, const void *B, void *C, int32_t M, int32_t N, int32_t K, int out_f32,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * Where the tensor-core sweep of the last kmip_attn_forward call on `workspace` put each query row,
 * so that tests can sample rows by their place in the sweep (work-item borders, the split tail of
 * the schedule) and not only by their row number.  Synchronises `stream`, then writes to HOST memory
 *   order[s]       = row number of the node the sweep handled at position s, s = 0 .. N-1
 *                    (the identity where the library keeps the row order: small problems, fp32 mode,
 *                    graphs below 8192 nodes);
 *   *rows_per_item = query rows per work item (128 x the query tiles a CTA owns; 128 in fp32 mode).
 * N, G, H, d, k, mode: as passed to that forward call.  Errors as for kmip_attn_workspace_bytes,
 * KMIP_ERR_CUDA if the synchronisation or the copy fails.
 */
int kmip_test_sweep_order(const void *workspace, int64_t N, int32_t G, int32_t H, int32_t d,
                          int32_t k, int mode, int32_t *order, int32_t *rows_per_item, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* KMIP_TEST_H_ */
