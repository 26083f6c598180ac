/*
 * dsmoe -- the DS-MoE feed-forward layer at inference, for NVIDIA B200 (sm_100a).
 *
 * One Mixture-of-Experts FFN layer as the paper states it (Section 3.1, Eq. 1):
 *
 *     S = softmax(h(X)),      O = sum_{i=1..K} S_{A_i} * e_{A_i}(X)
 *
 * with N experts e (MLPs with GeLU, "Model Hyperparameters" paragraph), a router h,
 * and A the indices of the K highest-scoring experts.  At inference K is either fixed
 * or set per token by how many experts score above a threshold eps ("Sparse Inference"
 * paragraph); the threshold is on the normalised probability S*N and must be exceeded
 * (Section 4.2 and its footnote).  The dense-training forward evaluates every expert
 * and weights it by its score ("Dense Training" paragraph, the forward behind Eq. 3);
 * here it is DSMOE_SELECT_ALL.
 *
 * Notation: T tokens in the call, d = model width (paper d_h / D_emb), E = number of
 * experts (paper N, N_ffd), H = hidden width of one expert (paper D_ffd),
 * k_t = number of experts selected for token t, A = sum_t k_t assignments.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, row-major, 16-byte
 *     aligned.  Nothing is allocated or freed by the library; nothing synchronises
 *     the host.  Work is enqueued on the caller's stream.
 *   - `desc` is a HOST pointer, read during the call only.
 *   - Return value: DSMOE_OK or an error; on error nothing has been enqueued unless the
 *     code is DSMOE_ERR_CUDA (a launch failed part-way).
 *   - Limits: 1 <= E <= 64, d % 8 == 0, H % 8 == 0, T >= 0 (T == 0 is a no-op).
 *     Violations return DSMOE_ERR_INVALID_ARG / DSMOE_ERR_UNSUPPORTED.
 *   - Inputs must be finite; NaN/Inf give unspecified values, never a fault.
 *   - dtype selects the storage type of x, W1, W2, xp, yp and out (fp32 or bf16).
 *     Router weights, scores and gates are always fp32; accumulation is fp32.
 *   - Amax = T*E for THRESHOLD and ALL, T*min(K,E) for TOPK: the capacity of every
 *     per-assignment buffer, so the data-dependent A never has to reach the host.
 *   - W = E for THRESHOLD and ALL, min(K,E) for TOPK: row stride of token_rows.
 *   - Host side: one thread at a time may call into the library (it keeps small per-device and
 *     per-buffer caches without locks).  Any number of devices may be used from that thread; a call
 *     works on the current device, which must own every pointer passed.
 */
#ifndef DSMOE_H_
#define DSMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DSMOE_OK = 0,
    DSMOE_ERR_INVALID_ARG = 1,   /* null pointer, bad shape, bad alignment, bad enum       */
    DSMOE_ERR_UNSUPPORTED = 2,   /* valid but outside the limits above (e.g. E > 64)       */
    DSMOE_ERR_WORKSPACE = 3,     /* ws_bytes smaller than dsmoe_workspace_size reports     */
    DSMOE_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                      */
    DSMOE_ERR_TIMEOUT = 5        /* written to *dev_status by a kernel whose bounded wait ran out */
} dsmoe_status;

typedef enum { DSMOE_F32 = 0, DSMOE_BF16 = 1 } dsmoe_dtype;

typedef enum {
    DSMOE_SELECT_THRESHOLD = 0,  /* expert e active iff score exceeds eps                  */
    DSMOE_SELECT_TOPK = 1,       /* the K highest scores; ties go to the lower index       */
    DSMOE_SELECT_ALL = 2,        /* every expert: the dense-training forward               */
    /* "Expert Sampling Strategy" paragraph, Threshold-TopK: the threshold rule gives each token a count of
     * active experts; the average count over the T tokens of the call, rounded half up and kept within
     * [1, E] (the paper leaves the rounding open), is the K of a top-K selection applied to every token.
     * eps and eps_normalized as for DSMOE_SELECT_THRESHOLD; K is ignored.  dsmoe_select_static does not
     * offer this mode (DSMOE_ERR_UNSUPPORTED). */
    DSMOE_SELECT_THRESHOLD_TOPK = 3
} dsmoe_mode;

typedef struct {
    int32_t T, d, H, E;
    int32_t dtype;            /* dsmoe_dtype                                               */
    int32_t mode;             /* dsmoe_mode                                                */
    float   eps;              /* THRESHOLD only                                            */
    int32_t eps_normalized;   /* 1: compare S*E > eps (the paper's normalised probability,
                                 one fp32 multiply); 0: compare S > eps                    */
    int32_t K;                /* TOPK only; K > E behaves as K = E                         */
    int32_t min_k;            /* 0: a token may select nothing and then outputs 0;
                                 1: such a token keeps its lowest-index argmax             */
    int32_t out_fp32;         /* 1: `out` is fp32 even when dtype is bf16                  */
    int32_t fuse_combine;     /* dsmoe_layer_forward with packed weights and a sparse selection -- where
                                 Eq. 1's sum over a token's experts is taken.  Either way each expert
                                 output is multiplied by its gate in fp32 in the down-projection's
                                 epilogue and nothing is rounded before the sum; the sum runs in
                                 ascending expert order and is bit-reproducible from run to run.
                                 1: inside the down-projection: its epilogue adds gate * output to the
                                    token's fp32 running sum; no expert outputs are stored, no second
                                    pass (least DRAM traffic; the read-modify-write of the sums goes
                                    through L2 and is hidden only when the experts are wide);
                                 2: the epilogue stores the gate-weighted outputs as fp32 rows and a
                                    second kernel adds a token's rows;
                                 0: the library chooses: 1 for a top-K selection with H >= 1024 and
                                    T*K >= 1024*E (wide experts, many row tiles per expert), else 2. */
} dsmoe_layer_desc;

/* A void* stands for the caller's cudaStream_t so that this header needs no CUDA include. */
typedef void* dsmoe_stream;

const char* dsmoe_status_string(dsmoe_status s);

/* Bytes of scratch for this desc.  A call takes one of two kinds of path, and their buffers overlap:
 * the plain path (fp32 layers, or no packed weights: grouped copy of the tokens, fp32 hidden
 * activations, expert outputs) and the tensor-core paths (packed bf16 weights: bf16 hidden activations
 * and an fp32 running sum of [T,d]).
 *   dsmoe_workspace_size         enough for any call with this desc (the larger of the two)
 *   dsmoe_workspace_size_packed  enough for dsmoe_expert_mlp / dsmoe_layer_forward when `packed` is
 *                                given (DSMOE_ERR_UNSUPPORTED if this desc has no tensor-core path)
 *   dsmoe_workspace_size_stages  enough for dsmoe_select and dsmoe_permute (index scratch only)
 * Every entry point checks ws_bytes against the figure of the path it takes. */
dsmoe_status dsmoe_workspace_size(const dsmoe_layer_desc* desc, size_t* bytes);
dsmoe_status dsmoe_workspace_size_packed(const dsmoe_layer_desc* desc, size_t* bytes);
dsmoe_status dsmoe_workspace_size_stages(const dsmoe_layer_desc* desc, size_t* bytes);

/*
 * Router scores, Eq. 1 (first half): scores[t,:] = softmax(x[t,:].Wr + br) over all E
 * experts, fp32 with the row maximum subtracted.
 *   x [T,d] dtype; Wr [d,E] fp32; br [E] fp32 or NULL; scores [T,E] fp32 (written).
 */
dsmoe_status dsmoe_router(const dsmoe_layer_desc* desc, const void* x, const float* Wr,
                          const float* br, float* scores, dsmoe_stream stream);

/*
 * Expert selection ("Sparse Inference" paragraph; Section 4.2 footnote), decided in fp32
 * on the given scores, so identical scores give bit-identical results everywhere.
 *   scores [T,E] fp32 (read); mask [T] uint64, bit e set iff expert e is selected;
 *   k_t [T] int32 = popcount(mask); counts [E] int32 = tokens per expert;
 *   offsets [E+1] int32 = exclusive prefix sum of counts, offsets[E] = A.
 * All four outputs are written in full.  workspace: at least dsmoe_workspace_size_stages bytes.
 */
dsmoe_status dsmoe_select(const dsmoe_layer_desc* desc, const float* scores, uint64_t* mask,
                          int32_t* k_t, int32_t* counts, int32_t* offsets, void* workspace,
                          size_t ws_bytes, dsmoe_stream stream);

/*
 * dsmoe_select without a workspace argument, for callers that cannot allocate device memory (code
 * that runs under a framework's own allocator, plugins given only their input and output buffers,
 * loops in which an allocation is not allowed).  The paper has no counterpart to this entry point:
 * it computes exactly what dsmoe_select computes, with the same arguments and results, but keeps
 * its scratch in a 512 KiB device array built into the library (held by every GPU that loads the
 * library, until the process exits).
 *   Limit: ceil(T/32) * E <= 131072 (e.g. T <= 65536 at E = 64, T <= 131072 at E = 32); beyond it
 *   the call returns DSMOE_ERR_WORKSPACE and nothing is enqueued -- use dsmoe_select.
 *   The first call on each device looks up the array's device address (with that device current);
 *   make that first call before starting any stream capture.
 *   It calls no allocation routine.  All calls on a device share the one array: calls whose kernels
 *   may overlap on the GPU (different streams) race on it and must be serialised by the caller.
 */
dsmoe_status dsmoe_select_static(const dsmoe_layer_desc* desc, const float* scores, uint64_t* mask,
                                 int32_t* k_t, int32_t* counts, int32_t* offsets, dsmoe_stream stream);

/*
 * Grouping of tokens by expert -- the token duplication the "GPU Inference Analysis"
 * section names.  Row r in [offsets[e], offsets[e+1]) holds the token with the
 * (r - offsets[e])-th smallest index among those that selected e.
 *   x [T,d] dtype, scores [T,E], mask [T], offsets [E+1]: read.
 *   row_token [Amax] int32: token of row r;  row_gate [Amax] fp32: scores[token,e];
 *   token_rows [T,W] int32: rows of token t in ascending expert order, -1 beyond k_t;
 *   xp [Amax,d] dtype: xp[r,:] = x[row_token[r],:].  Entries at r >= A are not written.
 *   workspace: at least dsmoe_workspace_size_stages bytes.  A row index that falls outside
 *   [0, Amax) because the given offsets do not belong to the given mask is skipped, never stored to.
 */
dsmoe_status dsmoe_permute(const dsmoe_layer_desc* desc, const void* x, const float* scores,
                           const uint64_t* mask, const int32_t* offsets, int32_t* row_token,
                           float* row_gate, int32_t* token_rows, void* xp, void* workspace,
                           size_t ws_bytes, dsmoe_stream stream);

/*
 * The selected experts' MLPs on grouped rows (Eq. 1's e(X); GeLU is the exact erf form):
 * yp[r,:] = GeLU(xp[r,:].W1[e]).W2[e] for r in [offsets[e], offsets[e+1]).
 *   xp [Amax,d] dtype; W1 [E,d,H] dtype; W2 [E,H,d] dtype; offsets [E+1]: read.
 *   yp [Amax,d] dtype (written for r < A).
 *   packed: NULL, or the buffer dsmoe_pack_weights filled from these W1, W2 (bf16 only);
 *   with it the tensor-core kernels run, without it a plain fp32-FMA kernel does.
 *   dev_status: optional device int32.  The tensor-core kernels check the segments first: an expert
 *   whose [offsets[e], offsets[e+1]) is negative, decreasing or ends beyond Amax is treated as empty
 *   (none of its rows is written) and DSMOE_ERR_INVALID_ARG is stored there; DSMOE_ERR_TIMEOUT if a
 *   bounded wait ran out.
 */
dsmoe_status dsmoe_expert_mlp(const dsmoe_layer_desc* desc, const void* xp, const void* W1,
                              const void* W2, const void* packed, const int32_t* offsets,
                              void* yp, void* workspace, size_t ws_bytes, int32_t* dev_status,
                              dsmoe_stream stream);

/*
 * Aggregation of expert outputs back into token order (Eq. 1's sum; the aggregation the
 * "GPU Inference Analysis" section names): out[t,:] = sum_i row_gate[r_i] * yp[r_i,:]
 * over r_i = token_rows[t,i], i < k_t[t], accumulated in fp32 in that order and rounded
 * once.  A token with k_t = 0 gets zeros.
 *   yp [Amax,d] dtype; row_gate [Amax]; token_rows [T,W]; k_t [T]: read.
 *   out [T,d] dtype (fp32 if desc->out_fp32).
 */
dsmoe_status dsmoe_combine(const dsmoe_layer_desc* desc, const void* yp, const float* row_gate,
                           const int32_t* token_rows, const int32_t* k_t, void* out,
                           dsmoe_stream stream);

/*
 * Kernel-preferred copy of the (static, post-training) expert weights, bf16: W1 as
 * [E][d/64][H][64] followed by W2 as [E][H/64][d][64] (block-major along the reduction), so
 * that every tensor-core operand is contiguous along the reduction and every tile a kernel
 * fetches is one contiguous piece of memory.  dtype must be DSMOE_BF16; d and H multiples of 64.
 * dsmoe_packed_size reports the bytes `packed` must hold.
 */
dsmoe_status dsmoe_packed_size(const dsmoe_layer_desc* desc, size_t* bytes);
dsmoe_status dsmoe_pack_weights(const dsmoe_layer_desc* desc, const void* W1, const void* W2,
                                void* packed, dsmoe_stream stream);

/*
 * The whole layer, Eq. 1: router -> selection -> grouping -> experts -> combine, or, for
 * DSMOE_SELECT_ALL, the dense-training forward  out = sum_e S_e * e_e(x).
 *   x [T,d]; Wr [d,E]; br [E] or NULL; W1 [E,d,H]; W2 [E,H,d]; packed NULL or from
 *   dsmoe_pack_weights (W1/W2 may then be NULL); out [T,d] dtype (fp32 if out_fp32).
 *   mask_out [T] uint64 and counts_out [E] int32: optional copies of the selection.
 *   dev_status: optional device int32; kernels write a dsmoe_status there if a bounded
 *   wait runs out or an index check fails (they then exit cleanly); untouched otherwise.
 *   With packed weights and a sparse selection the gate multiply sits in the down-projection's
 *   epilogue (fp32, before any rounding); desc->fuse_combine chooses whether the sum over a token's
 *   experts does too.
 */
dsmoe_status dsmoe_layer_forward(const dsmoe_layer_desc* desc, const void* x, const float* Wr,
                                 const float* br, const void* W1, const void* W2,
                                 const void* packed, void* out, uint64_t* mask_out,
                                 int32_t* counts_out, void* workspace, size_t ws_bytes,
                                 int32_t* dev_status, dsmoe_stream stream);

/*
 * Same call with HOST buffers for x and out (pinned or pageable): copies x to the device,
 * runs dsmoe_layer_forward, copies out back and waits for the stream.  x_dev [T,d] and
 * out_dev [T,d] are device staging buffers supplied by the caller.
 */
dsmoe_status dsmoe_layer_forward_host(const dsmoe_layer_desc* desc, const void* x_host,
                                      void* x_dev, const float* Wr, const float* br,
                                      const void* W1, const void* W2, const void* packed,
                                      void* out_dev, void* out_host, void* workspace,
                                      size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream);

/*
 * The same without the final wait: both copies and the layer are enqueued on `stream` and the call
 * returns.  x_host must stay unchanged and out_host unread until the caller has waited for the stream
 * (or an event recorded behind the call).  Calls on different streams, each with its own x_dev,
 * out_dev, out_host, workspace and dev_status, overlap one call's copies with another call's kernels:
 * the serving loop's form.  With pageable host buffers the copies wait by themselves.
 */
dsmoe_status dsmoe_layer_forward_host_async(const dsmoe_layer_desc* desc, const void* x_host,
                                            void* x_dev, const float* Wr, const float* br,
                                            const void* W1, const void* W2, const void* packed,
                                            void* out_dev, void* out_host, void* workspace,
                                            size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream);

/*
 * Selection statistics for logging ("Layer Utilization" paragraph: active experts per layer and per
 * token; Section 4.2 footnote for the threshold).  Written to the DEVICE struct `stats`:
 *   assignments     A = sum_t k_t                          zero_tokens    tokens that selected no expert
 *   counts[e]       tokens that selected expert e          empty_experts  experts selected by no token
 *   near_threshold  threshold rules only: how many scores lie within 1e-6 of eps (in the quantity the
 *                   rule compares: S, or fl32(S*E) when eps_normalized) -- decisions that a different
 *                   rounding of the softmax could flip; 0 for the other rules
 *   scores [T,E], mask [T]: read.  The caller copies the struct back when it wants the figures.
 */
typedef struct {
    int64_t assignments;
    int64_t near_threshold;
    int32_t zero_tokens;
    int32_t empty_experts;
    int32_t counts[64];
} dsmoe_selection_stats;

dsmoe_status dsmoe_stats(const dsmoe_layer_desc* desc, const float* scores, const uint64_t* mask,
                         dsmoe_selection_stats* stats, dsmoe_stream stream);

/*
 * Mutual-information loss of the router ("Mutual Information Loss" paragraph, Eq. 4-6) over the T tokens of
 * the call, natural logarithms:  p(e_i) = mean_t scores[t,i];  H(e) = -sum_i p(e_i) log p(e_i);
 * H(e|X_t) = -sum_i scores[t,i] log scores[t,i];  L_MI = -H(e) + mean_t H(e|X_t).
 *   scores [T,E] fp32: read.  loss3 [3] fp32 (device): L_MI, H(e), mean_t H(e|X_t).
 *   grad [T,E] fp32 or NULL: dL_MI/dscores[t,i] = (log p(e_i) - log scores[t,i]) / T.
 *   Sums are taken in double precision in a fixed order (bit-reproducible).  T >= 1.
 *   workspace: at least dsmoe_workspace_size_stages bytes.
 */
dsmoe_status dsmoe_mi_loss(const dsmoe_layer_desc* desc, const float* scores, float* loss3, float* grad,
                           void* workspace, size_t ws_bytes, dsmoe_stream stream);

/*
 * Gradients of dense training ("Dense Training" paragraph, Eq. 3) for a given gradient dO of the layer
 * output:  grad S_j = <e_j(X), dO> for every expert j, and grad e_j(X) = S_j dO, which is returned one
 * linear step further down, at the expert's hidden activation a_j = GeLU(X.W1[j]) (e_j(X) = a_j.W2[j]):
 * dA[t, j*H + k] = S_j * sum_c dO[t,c] * W2[j][k,c].  With mask (Eq. 2, sparse training: M marks the experts
 * that were active in the forward pass) both are zero for the other experts.  Activations are recomputed
 * from x (nothing of the forward pass has to be kept).
 *   x [T,d], dO [T,d] dtype; W1 [E,d,H], W2 [E,H,d] dtype; scores [T,E] fp32; mask [T] uint64 or NULL: read.
 *   dS [T,E] fp32; dA [T,E*H] dtype: written.
 *   packed: NULL, or the buffer dsmoe_pack_weights filled from these weights (bf16): then the tensor cores
 *   run (W1 may be NULL, W2 is still read in its natural layout) and the workspace must hold
 *   dsmoe_workspace_size_packed bytes; without it a plain fp32-FMA kernel runs and needs no workspace.
 */
dsmoe_status dsmoe_dense_backward(const dsmoe_layer_desc* desc, const void* x, const void* W1, const void* W2,
                                  const void* packed, const float* scores, const uint64_t* mask, const void* dO,
                                  float* dS, void* dA, void* workspace, size_t ws_bytes, int32_t* dev_status,
                                  dsmoe_stream stream);

/*
 * The mixture-of-attention-heads layer ("Mixture of Attention Head" paragraph, Eq. 7-8): the model's other MoE
 * block.  Expert i owns n_head query heads and their output projections; keys and values are shared by all experts,
 * head j of every expert attending to key/value head j.  For token t, which sees keys 0..pos[t] of its sequence's cache:
 *
 *   Q_ij = x_t . Wq[i][:, j*dh:(j+1)*dh]              a_ij = softmax_l(scale <Q_ij, K[seq][j][l]>) . V[seq][j]
 *   O_t  = sum over the selected experts i (ascending) of S[t,i] * sum_j a_ij . Wo[i][j*dh:(j+1)*dh, :]
 *
 * It is the feed-forward layer's pipeline with attention in place of GeLU: desc describes it with E = the number of
 * attention experts and H = n_head * d_head; router, selection (desc->mode ...), grouping and the router-weighted sum
 * are those of dsmoe_layer_forward.  Eq. 7 prints no scale under the softmax: `scale` is the caller's (1/sqrt(d_head)
 * in the usual form).  No biases.  Queries and attention outputs are rounded to bf16 between the steps.
 *
 * args (host struct, read during the call): Kc, Vc  device, bf16 [n_seq][n_head][L][d_head]; tok_seq  device int32 [T],
 * the sequence of each token, or NULL (all 0); pos  device int32 [T], 0 <= pos[t] < L.
 * packed   device: dsmoe_pack_weights(desc, Wq, Wo, packed) with Wq [E][d][H], Wo [E][H][d].
 * x, Wr, br, out, mask_out, counts_out, workspace (dsmoe_workspace_size_packed(desc) bytes), dev_status: as for
 * dsmoe_layer_forward.  Supported: bf16, d and H multiples of 64, d_head 64, 96 or 128 (any L), or another
 * multiple of 32 up to 256 with L up to 12000; DSMOE_ERR_UNSUPPORTED otherwise.  A tok_seq or pos entry out of range is clamped and reported as
 * DSMOE_ERR_INVALID_ARG in *dev_status.
 */
typedef struct dsmoe_moa_args {
    int32_t n_head, n_seq, L;
    float scale;
    const void* Kc;
    const void* Vc;
    const int32_t* tok_seq;
    const int32_t* pos;
} dsmoe_moa_args;
dsmoe_status dsmoe_moa_forward(const dsmoe_layer_desc* desc, const dsmoe_moa_args* args, const void* x, const float* Wr,
                               const float* br, const void* packed, void* out, uint64_t* mask_out, int32_t* counts_out,
                               void* workspace, size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream);

/*
 * Measurement aid (no counterpart in the paper): a ring of CUDA event pairs on the caller's stream.
 * After dsmoe_timing_enable(n_pairs) (n_pairs > 0; events are created here, so call it outside any
 * timed region), every launch of an expert-MLP tensor-core kernel (the two grouped or dense GEMMs of
 * a prefill call, the one kernel of a decode call) is bracketed by the next pair until n_pairs are
 * used.  dsmoe_timing_read waits for the recorded pairs, writes their durations in milliseconds, in
 * launch order, to the HOST array ms (at most n_max), sets *n and empties the ring.
 * dsmoe_timing_enable(0) switches it off.  Off by default.
 */
dsmoe_status dsmoe_timing_enable(int n_pairs);
dsmoe_status dsmoe_timing_read(float* ms, int n_max, int* n);

#ifdef __cplusplus
}
#endif
#endif /* DSMOE_H_ */
