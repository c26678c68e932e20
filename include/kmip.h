/*
 * kmip.h -- C ABI of the B200 (sm_100a) k-Maximum-Inner-Product self-attention library.
 *
 * The library computes the hot path of multi-head k-MIP self-attention (Eq. 1-2 and
 * Algorithm 1, lines 2-6, of "k-Maximum Inner Product Attention for Graph Transformers")
 * and its sparse backward pass (Sec. 3.1: the top-k indices are reused, the search is
 * not repeated), for a batch of graphs stored back to back and delimited by CSR offsets.
 *
 * Conventions shared by every call
 *   N        total number of nodes of the batch (all graphs concatenated), 0 <= N < 2^31
 *   G        number of graphs; graph g owns rows graph_offsets[g] .. graph_offsets[g+1]-1
 *   H, d, k  heads, per-head width (d_K = d_V = d), keys kept per query
 *   layouts  Q, K, V, out, d_out, dQ, dK, dV : [N, H, d] row-major (a node's H*d values are
 *            contiguous, head h at columns h*d .. h*d+d-1);
 *            topk_idx : int32 [N, H, k];  topk_score : float [N, H, k];
 *            graph_offsets : int32 [G+1], offsets[0] = 0, non-decreasing, offsets[G] = N.
 *   memory   every pointer is DEVICE memory owned by the caller, 16-byte aligned, and stays
 *            valid until the work enqueued on `stream` has finished.  The library allocates
 *            no device memory and keeps no state between calls, with two documented exceptions:
 *            kmip_attn_forward_static_scratch (a built-in scratch array and its cached device
 *            address) and the kmip_profile_* calls (process-wide CUDA events).  `workspace` is
 *            caller-owned scratch whose contents are undefined between calls.  Its first 256
 *            bytes are a status block that kmip_last_status reads.
 *   async    calls validate their arguments on the host, enqueue kernels on `stream`
 *            (a cudaStream_t passed as void*, NULL = default stream) and return without
 *            synchronising.  KMIP_OK means "enqueued".  Problems only the device can see
 *            (malformed offsets, an expired bounded wait) are recorded in the status block;
 *            the kernels enqueued after such a problem return without writing, so the call's
 *            outputs are undefined whenever the status word is not KMIP_OK.
 *   errors   nothing is enqueued when a call returns a status other than KMIP_OK.
 */
#ifndef KMIP_H_
#define KMIP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KMIP_OK = 0,
    KMIP_ERR_INVALID_ARG = 1,  /* null or misaligned pointer, negative size, k < 1, H < 1, N*H*k >= 2^31 */
    KMIP_ERR_UNSUPPORTED = 2,  /* d not in {16, 32, 64, 128}, k > 128, unknown mode */
    KMIP_ERR_WORKSPACE = 3,    /* workspace smaller than kmip_attn_workspace_bytes reports */
    KMIP_ERR_CUDA = 4,         /* a CUDA runtime call or a kernel launch failed */
    KMIP_ERR_TIMEOUT = 5,      /* device side: a bounded wait inside a kernel ran out */
    KMIP_ERR_BAD_OFFSETS = 6,  /* device side: graph_offsets is not a valid CSR row-pointer array */
    KMIP_ERR_TOO_LARGE = 7,    /* kmip_attn_forward_static_scratch: the problem needs more than the built-in scratch */
    KMIP_ERR_CHECK = 8         /* device side, only in a library built with -DKMIP_CHECKS: an index test failed or a
                                  canary block between two workspace regions was overwritten */
} kmip_status_t;

typedef enum {
    /* Q, K, V, out, d_out, dQ, dK, dV hold bf16.  Scores are a dense bf16 contraction with fp32
       accumulation on the tcgen05 tensor cores; softmax, sums and gradients accumulate in fp32. */
    KMIP_BF16_TC = 0,
    /* All of them hold fp32.  Scores are fp32 fused multiply-adds in index order c = 0..d-1. */
    KMIP_FP32_EXACT = 1,
    /* KMIP_BF16_TC with an exact pruning of the search (the quadratic search is the first limitation the
       paper names, Sec. 6): in graphs of 8192 nodes or more the keys are swept in an order that puts heavy
       and similar keys together, and a 128-key tile is skipped for a block of query rows when a bound on
       every inner product of the pair (centroids and radii, or Cauchy-Schwarz with the largest key norm)
       lies below all of the block's current k-th best scores.  Same results as KMIP_BF16_TC up to the
       order in which equal scores are met; forward only differs, the backward pass is the same.
       Needs about 16 more bytes per node, 4 per (node, head) and (d + 4) * 4 * H per 128 nodes of scratch.
       Below 32768 nodes it is KMIP_BF16_TC. */
    KMIP_BF16_TC_PRUNED = 2
} kmip_mode_t;

#define KMIP_PASS_FORWARD 0
#define KMIP_PASS_BACKWARD 1

/*
 * Scratch size in bytes that kmip_attn_forward (pass = 0) or kmip_attn_backward (pass = 1)
 * needs for this problem size.  Linear in N*H*(k + d): the N x N score matrix of Algorithm 1
 * line 2 is never stored (Sec. 3.1, App. F).  Forward: one bf16 copy of K regrouped by head and, from
 * 32768 nodes on, one of Q in the sweep's row order plus 6 bytes per node
 * (tensor-core mode only), for head widths up to 32 and k <= 32 also 6 bytes per kept candidate group
 * (16, 24 or 48 per (node, head)), plus the work list; backward: 40 bytes per selected pair, 12 bytes per
 * (node, head) and a table of digit counts of the sort that builds the hit lists (at most 4 bytes per
 * selected pair, 1 to 2 at the sizes of the paper's experiments).  Host only, no CUDA call.
 */
int kmip_attn_workspace_bytes(int64_t N, int32_t G, int32_t H, int32_t d, int32_t k,
                              int mode, int pass, size_t *bytes);

/*
 * Forward pass, Eq. 1 and Algorithm 1 lines 2-6, for every head h and every query node i:
 *   s_ij       = q_i^h . k_j^h   for all nodes j of i's own graph (self included)
 *   topk       : the k largest s_ij; ties go to the lower j; listed by (score desc, j asc)
 *   topk_idx   = their global row numbers j        (I_argtopk of Algorithm 1 line 3)
 *   topk_score = their raw inner products s_ij     (E_topk; the 1/sqrt(d) factor is not applied here)
 *   out[i,h,:] = sum_t softmax_t(topk_score / sqrt(d)) * V[topk_idx_t, h, :]   (lines 4-6)
 * A graph with n < k nodes keeps all n and pads: topk_idx = -1, topk_score = -inf, weight 0.
 * graph_offsets may be NULL, meaning one graph [0, N) (G is then ignored).
 * N = 0 returns KMIP_OK and enqueues nothing.
 * Inputs: Q, K, V, graph_offsets.  Outputs (fully overwritten when the device status word stays
 * KMIP_OK, undefined otherwise): out, topk_idx, topk_score.
 * In KMIP_BF16_TC mode the selection uses tensor-core scores, so a key whose exact score
 * differs from the k-th best by less than the fp32 accumulation error may swap with it.
 */
int kmip_attn_forward(const void *Q, const void *K, const void *V,
                      const int32_t *graph_offsets, int32_t G, int64_t N,
                      int32_t H, int32_t d, int32_t k, int mode,
                      void *out, int32_t *topk_idx, float *topk_score,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward pass through Algorithm 1 lines 4-6 with the selection held constant (Sec. 3.1,
 * App. E: I_argtopk and E_topk are reused).  With p = softmax(topk_score / sqrt(d)) and
 * upstream gradient g = d_out:
 *   dP_t = g_i . v_{j_t}     D = sum_t p_t dP_t     dS_t = p_t (dP_t - D) / sqrt(d)
 *   dQ[i,h,:] = sum_t dS_t K[j_t,h,:]
 *   dK[m,h,:] = sum over (i,t) with j_t = m of dS_t Q[i,h,:]
 *   dV[m,h,:] = sum over (i,t) with j_t = m of p_t g[i,h,:]
 * Slots with topk_idx < 0 are ignored; keys nobody selected get zero gradient.
 * Inputs: Q, K, V, d_out, topk_idx, topk_score as written by kmip_attn_forward on the same
 * Q, K; `out` is accepted for symmetry with autograd interfaces and may be NULL.
 * Outputs (fully overwritten): dQ, dK, dV.  graph_offsets and G are not needed by the
 * arithmetic (indices are global) and may be NULL / 0.
 * dK and dV are sums over each key's list of hits in query order (the lists are built by a stable sort,
 * without atomics), so the same inputs give the same gradients bit for bit on every run (up to 2^24
 * (node, head) pairs and 2^31 selected pairs; beyond that the lists are filled with atomic counters and
 * the sums are reproducible to fp32 rounding only).
 */
int kmip_attn_backward(const void *Q, const void *K, const void *V,
                       const int32_t *graph_offsets, int32_t G, int64_t N,
                       int32_t H, int32_t d, int32_t k, int mode,
                       const void *out, const void *d_out,
                       const int32_t *topk_idx, const float *topk_score,
                       void *dQ, void *dK, void *dV,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * Training variants with attention dropout on the k softmax weights (the paper trains its LRGB and
 * City-Networks models with attention dropout 0.5 and its point-cloud models with 0; App. H).
 * Each weight p_t of Algorithm 1 line 5 is kept with probability 1 - drop_p and divided by
 * 1 - drop_p, independently per (query, head, slot):
 *   out[i,h,:] = sum_t f_t p_t V[topk_idx_t, h, :],   f_t = 1/(1 - drop_p) or 0.
 * The draws are counter based, so the backward call regenerates them from the same (drop_p, seed)
 * and nothing is stored: slot t of query i, head h uses the ((i*H + h)*k + t + 1)-th output of
 * SplitMix64 started at `seed`; its top 24 bits / 2^24 is the uniform, kept when >= drop_p.
 * topk_idx and topk_score are not affected.  In the backward pass f is a constant:
 *   dP_t = f_t (g_i . v_{j_t}),  dV gets f_t p_t g_i,  D, dS, dQ, dK as in kmip_attn_backward.
 * drop_p must be in [0, 1) (else KMIP_ERR_INVALID_ARG); drop_p = 0 is exactly kmip_attn_forward /
 * kmip_attn_backward.  All other arguments, layouts, ownership and errors are theirs.
 */
int kmip_attn_forward_dropout(const void *Q, const void *K, const void *V,
                              const int32_t *graph_offsets, int32_t G, int64_t N,
                              int32_t H, int32_t d, int32_t k, int mode,
                              float drop_p, uint64_t seed,
                              void *out, int32_t *topk_idx, float *topk_score,
                              void *workspace, size_t workspace_bytes, void *stream);
int kmip_attn_backward_dropout(const void *Q, const void *K, const void *V,
                               const int32_t *graph_offsets, int32_t G, int64_t N,
                               int32_t H, int32_t d, int32_t k, int mode,
                               float drop_p, uint64_t seed,
                               const void *out, const void *d_out,
                               const int32_t *topk_idx, const float *topk_score,
                               void *dQ, void *dK, void *dV,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * Diagnostic of the paper's App. I (cumulative attention weight): for every query node and head,
 * the share of the FULL softmax over all nodes of its graph that falls on the k keys kept by the
 * forward pass,
 *   mass[i,h] = sum_t exp(topk_score[i,h,t] / sqrt(d)) / sum_j exp(q_i^h . k_j^h / sqrt(d)),
 * a number in (0, 1]; 1 when the graph has at most k nodes.  It needs every score of the row once more.
 * In the bf16 modes they come from the tensor cores (the pipeline of the forward sweep with a running
 * log-sum-exp in place of the selection: about the cost of one forward sweep, every head width); in
 * KMIP_FP32_EXACT mode they are fp32 sums on CUDA cores, about ten times slower, d = 128 not supported
 * there (KMIP_ERR_UNSUPPORTED).  Meant for inspection, not for the training loop.
 * Inputs: Q, K, graph_offsets as for kmip_attn_forward; topk_score [N, H, k] as written by it.
 * Output (fully overwritten): mass, device memory, float [N, H], 4-byte aligned.
 * workspace: at least kmip_attn_workspace_bytes(..., KMIP_PASS_FORWARD) bytes; its contents are
 * overwritten, and its status block reports malformed offsets as for the forward pass.
 */
int kmip_attn_topk_mass(const void *Q, const void *K,
                        const int32_t *graph_offsets, int32_t G, int64_t N,
                        int32_t H, int32_t d, int32_t k, int mode,
                        const float *topk_score, float *mass,
                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * The full layer of Eq. 2 (Algorithm 1 with its "Require" line and line 8), bf16 tensor-core mode:
 *   Q^h = X W_Q^h,  K^h = X W_K^h,  V^h = X W_V^h,  O^h = kMIP-Attn(Q^h, K^h, V^h) inside each graph,
 *   Y = sum_h O^h W_O^h,
 * and its backward pass with the selection held constant (Sec. 3.1).  The four projections and every
 * product of the backward pass run on the tensor cores in the library's own kernels; the attention core
 * is kmip_attn_forward / kmip_attn_backward.  All tensors are bf16 device memory, 16-byte aligned:
 *   x [N, d_model];  w_q, w_k, w_v [H*d_head, d_model] (row h*d_head + c holds column c of W^h);
 *   w_o [d_model, H*d_head];  y, d_y, d_x [N, d_model];  dw_* in the shapes of the weights.
 * d_model must be a multiple of 8, 1 <= d_head <= 128, k <= 128.  A head width other than 16, 32, 64, 128 (the
 * paper's own study uses 10) is zero-padded to the next of those, d_pad, inside the call, which leaves
 * every inner product unchanged; the softmax still divides by sqrt(d_head).
 * Saved between the two calls, owned by the caller: q, k, v, o : bf16 [N, H, d_pad]; topk_idx int32 [N, H, k];
 * topk_score float [N, H, k] - written by kmip_layer_forward, read by kmip_layer_backward.
 * workspace: kmip_layer_workspace_bytes(..., pass) bytes of scratch; its first 256 bytes are the status
 * block kmip_last_status reads (device-side problems of the attention core are forwarded to it).
 * Errors, asynchrony and ownership as for kmip_attn_forward; other modes are KMIP_ERR_UNSUPPORTED.
 */
typedef struct {
    const void *x, *w_q, *w_k, *w_v, *w_o;   /* inputs */
    void *q, *k, *v, *o;                     /* saved projections and attention output, [N, H, d_pad] */
    int32_t *topk_idx;                       /* saved selection */
    float *topk_score;
    void *y;                                 /* forward output; unused by the backward pass */
    const void *d_y;                         /* backward input; unused by the forward pass */
    void *d_x, *dw_q, *dw_k, *dw_v, *dw_o;   /* backward outputs (fully overwritten) */
} kmip_layer_tensors_t;

int kmip_layer_workspace_bytes(int64_t N, int32_t G, int32_t d_model, int32_t H, int32_t d_head, int32_t k,
                               int pass, size_t *bytes);
int kmip_layer_forward(const kmip_layer_tensors_t *t, const int32_t *graph_offsets, int32_t G, int64_t N,
                       int32_t d_model, int32_t H, int32_t d_head, int32_t k,
                       void *workspace, size_t workspace_bytes, void *stream);
int kmip_layer_backward(const kmip_layer_tensors_t *t, const int32_t *graph_offsets, int32_t G, int64_t N,
                        int32_t d_model, int32_t H, int32_t d_head, int32_t k,
                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * Size in bytes of the scratch array that is built into the library for
 * kmip_attn_forward_static_scratch (8 MiB; each GPU that loads the library holds it until the
 * process exits).
 */
#define KMIP_STATIC_SCRATCH_BYTES ((size_t)8 << 20)

/*
 * The forward pass of kmip_attn_forward for callers that cannot provide a workspace because they
 * are not allowed to allocate device memory - for example a plug-in inside a framework that owns
 * all device memory, or a serving loop whose memory pool is frozen after start-up (an allocation
 * would also synchronise the device).  The paper has no counterpart; this is packaging only.
 * Same arguments, results and status codes as kmip_attn_forward, except:
 *   - there is no workspace argument: the scratch is a fixed KMIP_STATIC_SCRATCH_BYTES array inside
 *     the library.  A problem whose kmip_attn_workspace_bytes(..., KMIP_PASS_FORWARD) exceeds it is
 *     refused with KMIP_ERR_TOO_LARGE before anything is enqueued.  In tensor-core mode the scratch
 *     is dominated by one bf16 copy of K (and one of Q from 32768 nodes on), so the limit is about
 *     N*H*d <= 4.1 million elements (2 million from 32768 nodes on)
 *     (e.g. 32 000 nodes at H = 4, d = 32); fp32 mode needs 20 bytes per 128 nodes and per graph.
 *   - device_status (DEVICE pointer, may be NULL): if given, the device status word of this call
 *     (KMIP_OK, KMIP_ERR_TIMEOUT or KMIP_ERR_BAD_OFFSETS) is copied there on `stream` after the
 *     kernels, since there is no workspace for kmip_last_status to read (N = 0: KMIP_OK is
 *     stored there, nothing else is enqueued).
 *   - the call itself calls no cudaMalloc / cudaFree or any other allocating routine.  The first call
 *     on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - every call on a device uses the same array: two calls whose kernels can overlap on the GPU
 *     (different streams, or several host threads) race and give undefined results; calls on one
 *     stream are safe back to back.  The array keeps the last call's contents; each call clears or
 *     rewrites every part it reads.
 */
int kmip_attn_forward_static_scratch(const void *Q, const void *K, const void *V,
                                     const int32_t *graph_offsets, int32_t G, int64_t N,
                                     int32_t H, int32_t d, int32_t k, int mode,
                                     void *out, int32_t *topk_idx, float *topk_score,
                                     int32_t *device_status, void *stream);

/*
 * Synchronises `stream`, then copies the device status word of the last call that used
 * `workspace` into *device_status (KMIP_OK, KMIP_ERR_TIMEOUT or KMIP_ERR_BAD_OFFSETS).
 * Returns KMIP_ERR_CUDA if the synchronisation or the copy fails.  For tests and debugging;
 * not needed on the hot path.
 */
int kmip_last_status(const void *workspace, void *stream, int *device_status);

/*
 * Work counters of the last forward call on `workspace` (the paper has no counterpart).  Synchronises
 * `stream`, then reads from the status block of `workspace` into counters[8] (HOST memory, int64):
 *   [0..3]  KMIP_BF16_TC_PRUNED: key tiles of all work items, key tiles loaded (one end marker per work
 *           item included), (key tile, query tile) pairs, pairs scored, summed over the sweep's CTAs;
 *   [4]     KMIP_BF16_TC with d <= 32 and k <= 32: (query, head) pairs that the half-precision prefilter
 *           could not decide and the exact kernel recomputed from all keys;
 *   [5..7]  zero.
 * Counters of a path that did not run are zero.  Returns KMIP_ERR_CUDA if the synchronisation or the
 * copy fails.
 */
int kmip_attn_sweep_counters(const void *workspace, void *stream, int64_t *counters);

/*
 * Optional per-stage timing for benchmarks; the paper has no counterpart (its Fig. 3 reports a
 * stage breakdown measured from outside).  kmip_profile_enable(n > 0) creates CUDA events for up
 * to n forward and n backward calls (n <= 256) and makes the two passes record them around their
 * stages on the caller's stream; kmip_profile_enable(0) destroys them and turns recording off.
 * kmip_profile_read waits for the recorded events, adds up the stage times in milliseconds into
 * stage_ms[7] = {plan (+ key regrouping), score+select sweep, rescoring of the candidate groups,
 * softmax+gather-V, backward rows, inverse index, dK/dV segments}, stores the number of forward /
 * backward calls recorded in calls[2] and resets the counters.  Process-wide state, not thread-safe, one device; leave it off on the hot path.
 */
int kmip_profile_enable(int max_calls);
int kmip_profile_read(double *stage_ms, int *calls);

/* Static, NUL-terminated description of a status code. */
const char *kmip_status_string(int status);

/* Library version, major*10000 + minor*100 + patch. */
int kmip_version(void);

/*
 * Build flags of the loaded library: bit 0 is set in a -DKMIP_CHECKS build (libkmip_checks.so), which puts
 * 256-byte canary blocks between the regions of every workspace (kmip_attn_workspace_bytes of that library
 * already counts them), verifies them after each pass and tests indices before following them; problems
 * are reported as KMIP_ERR_CHECK in the status word, never by a trap.  Slower; for debugging and tests.
 */
int kmip_build_flags(void);

#ifdef __cplusplus
}
#endif
#endif /* KMIP_H_ */
