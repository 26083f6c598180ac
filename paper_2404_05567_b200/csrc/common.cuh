// Shared declarations of the dsmoe CUDA library: argument checks, the workspace layout and the
// internal launchers that the C entry points in api.cu call.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "dsmoe.h"

namespace dsmoe {

constexpr int kMaxExperts = 64;
constexpr int kChunk = 32;   // tokens per ballot chunk in the grouping kernels
constexpr int kSmallMaxT = 128;      // the small-T (decode) path keeps all tokens in one 128-row MMA tile
constexpr int kSmallMaxCtas = 192;   // upper bound on that path's grid (sizes its partial-sum buffer)

#define DSMOE_CUDA_TRY(expr)                                  \
    do {                                                      \
        cudaError_t err__ = (expr);                           \
        if (err__ != cudaSuccess) return DSMOE_ERR_CUDA;      \
    } while (0)

#define DSMOE_TRY(expr)                                       \
    do {                                                      \
        dsmoe_status st__ = (expr);                           \
        if (st__ != DSMOE_OK) return st__;                    \
    } while (0)

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

static inline size_t elem_size(int dtype) { return dtype == DSMOE_BF16 ? 2 : 4; }
static inline int width_of(const dsmoe_layer_desc& p) {
    return p.mode == DSMOE_SELECT_TOPK ? (p.K < p.E ? p.K : p.E) : p.E;
}
static inline size_t amax_of(const dsmoe_layer_desc& p) { return (size_t)p.T * (size_t)width_of(p); }

dsmoe_status check_desc(const dsmoe_layer_desc* desc);
static inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Byte offsets of every internal buffer inside the caller's workspace.  The small per-token and per-assignment
// index buffers come first (`stage_total` bytes: all that dsmoe_select and dsmoe_permute touch); the large
// activation buffers follow and overlap between the execution paths, of which a call takes exactly one:
//   plain (fp32-FMA GEMMs)     xp, h (fp32), yp
//   tensor-core paths          h (bf16: grouped [Amax,H]; dense and small-T [T,E*H]), acc (grouped: fp32 [T,d] running
//                              sum of the expert outputs), partial (small-T), router (split Wr, partial logits)
// total_packed = bytes a call with packed weights needs; total = the maximum over both kinds of call.
struct WsLayout {
    size_t scores, mask, k_t, counts, offsets, chunk_prefix, batch_k, sync, tile_done, mi, row_token, row_gate, token_rows;
    size_t stage_total;
    size_t xp, h_plain, yp;                 // plain path
    size_t h, acc, partial, router, bwd;    // tensor-core paths
    size_t total_plain, total_packed, total;
};
WsLayout ws_layout(const dsmoe_layer_desc& p);

// What the library keeps per device (attributes that must be set once per device, the SM count).  Entry points
// are not thread-safe: one host thread at a time may call into the library.
constexpr int kMaxDeviceSlots = 64;
struct DeviceState {
    int sm_count = 0;
    bool attr_gemm = false, attr_small = false, attr_router_f32 = false, attr_router_bf16 = false;
    int max_pairs = -1;   // CTA pairs of umma_gemm_kernel that can be resident at once; -1 not asked yet, 0 pairs unavailable
};
dsmoe_status device_state(DeviceState** out, int* device = nullptr);   // of the current device

// ---- router.cu
dsmoe_status launch_router(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                           float* scores, uint64_t* mask, int32_t* k_t, cudaStream_t s);
// k_scratch: one int of device memory, needed by DSMOE_SELECT_THRESHOLD_TOPK only (the batch's K)
dsmoe_status launch_select(const dsmoe_layer_desc& p, const float* scores, uint64_t* mask, int32_t* k_t,
                           cudaStream_t s, int* k_scratch = nullptr);
// launch_finalize = launch_chunk_counts (per chunk of 32 tokens, how many selected each expert) + launch_chunk_scan
// (prefixes over the chunks, counts, offsets)
dsmoe_status launch_chunk_counts(const dsmoe_layer_desc& p, const uint64_t* mask, int32_t* chunk_prefix, cudaStream_t s);
dsmoe_status launch_chunk_scan(const dsmoe_layer_desc& p, int32_t* counts, int32_t* offsets, int32_t* chunk_prefix,
                               int32_t* counts_out, cudaStream_t s);
dsmoe_status launch_finalize(const dsmoe_layer_desc& p, const uint64_t* mask, int32_t* counts,
                             int32_t* offsets, int32_t* chunk_prefix, int32_t* counts_out, cudaStream_t s);

// ---- permute.cu
// zero_out (optional): the layer output [T,d]; rows of tokens that selected no expert are set to zero
dsmoe_status launch_permute(const dsmoe_layer_desc& p, const void* x, const float* scores,
                            const uint64_t* mask, const int32_t* offsets, const int32_t* chunk_prefix,
                            int32_t* row_token, float* row_gate, int32_t* token_rows, void* xp,
                            cudaStream_t s, void* zero_out = nullptr);
// Grouping for the fused layers: counts, offsets and the row indices of launch_finalize + launch_permute (without a
// grouped copy of x).  chunk_counts_ready: chunk_prefix already holds the chunks' counts (the router wrote them).
dsmoe_status launch_group(const dsmoe_layer_desc& p, const float* scores, const uint64_t* mask, int32_t* counts,
                          int32_t* offsets, int32_t* chunk_prefix, int32_t* counts_out, int32_t* row_token,
                          float* row_gate, int32_t* token_rows, cudaStream_t s, void* zero_out, bool chunk_counts_ready);
// Selection statistics (see dsmoe_stats)
dsmoe_status launch_stats(const dsmoe_layer_desc& p, const float* scores, const uint64_t* mask,
                          dsmoe_selection_stats* stats, cudaStream_t s);
// yp_f32: the rows are fp32 whatever p.dtype says; row_gate == NULL: the rows are gate-weighted already
dsmoe_status launch_combine(const dsmoe_layer_desc& p, const void* yp, const float* row_gate,
                            const int32_t* token_rows, const int32_t* k_t, void* out, cudaStream_t s,
                            bool yp_f32 = false);
// Whether dsmoe_layer_forward's tensor-core grouped path aggregates inside the down-projection (see dsmoe.h)
// The library's own choice (fuse_combine == 0): inside only where it was measured to be as fast as the second
// kernel -- wide experts (a long enough mainloop to hide the read-modify-write of the sums) and a top-K selection
// with at least eight row tiles per expert on average (few tiles per expert make consecutive experts' tiles, which
// must take turns on the same sums, run at the same time).
static inline bool fuses_combine(const dsmoe_layer_desc& p) {
    if (p.fuse_combine != 0) return p.fuse_combine == 1;
    return p.mode == DSMOE_SELECT_TOPK && p.H >= 1024 && (long long)p.T * width_of(p) >= 1024ll * p.E;
}
dsmoe_status launch_pack(const dsmoe_layer_desc& p, const void* W1, const void* W2, void* packed,
                         cudaStream_t s);

// ---- mlp_generic.cu : plain fp32-FMA grouped GEMMs (any dtype, no packed weights needed)
dsmoe_status launch_mlp_generic(const dsmoe_layer_desc& p, const void* xp, const void* W1, const void* W2,
                                const int32_t* offsets, float* h, void* yp, cudaStream_t s);


// ---- mlp_umma.cu : tcgen05 / TMEM / TMA kernels on packed bf16 weights
dsmoe_status timing_enable(int n_pairs);
dsmoe_status timing_read(float* ms, int n_max, int* n);
bool umma_supported(const dsmoe_layer_desc& p);   // bf16, d and H multiples of 64
// Router for many tokens with the logits on the tensor cores (bf16 x; Wr split exactly into three bf16 terms, fp32
// accumulation), then softmax and selection.  `scratch` holds router_umma_scratch(p) bytes.
bool router_umma_supported(const dsmoe_layer_desc& p);
size_t router_umma_scratch(const dsmoe_layer_desc& p, size_t* split_bytes = nullptr);
dsmoe_status launch_router_umma(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                float* scores, uint64_t* mask, int32_t* k_t, char* scratch, int32_t* dev_status,
                                cudaStream_t s, int32_t* chunk_counts = nullptr);   // chunk_counts: see launch_group
// Grouped expert MLPs on expert-sorted rows: h = GeLU(xp.W1[e]) (bf16, in `hbuf`), yp = h.W2[e].
// With row_token (and x), the up-projection gathers its rows from x by index and xp is not read.
// With cmb->out, the down-projection's epilogue also aggregates (Eq. 1's weighted sum, ascending expert order per
// token): it writes the layer output cmb->out [T,d] and yp is not touched.  With cmb->out == NULL only the gate
// multiply moves into the epilogue: yp[r,:] = row_gate[r] * e(x)[r,:], stored as fp32.
struct CombineArgs {
    const int32_t* row_token;
    const float* row_gate;
    const uint64_t* mask;
    float* acc;          // fp32 [T,d] running sums (unused when the output itself is fp32)
    int* tile_done;      // E * ceil(d / 256) ints
    void* out;
};
// With moa, the layer is the mixture of attention heads (Eq. 7-8): the up-projection is the experts' query projection
// (no activation) and every grouped row attends to its sequence's keys and values before the down-projection.
struct MoaCore {
    int n_head, n_seq, L;
    float scale;
    const void* Kc;
    const void* Vc;          // [n_seq][n_head][L][d_head]
    const int32_t* tok_seq;  // [T] or NULL (one sequence)
    const int32_t* pos;      // [T]: token t sees keys 0..pos[t]
    const int32_t* token_rows;   // [T, W]: the grouped rows of each token (from the permute step)
};
dsmoe_status launch_mlp_umma(const dsmoe_layer_desc& p, const void* xp, const void* packed, const int32_t* offsets,
                             void* hbuf, void* yp, int32_t* dev_status, cudaStream_t s, const void* x = nullptr,
                             const int32_t* row_token = nullptr, const CombineArgs* cmb = nullptr,
                             const MoaCore* moa = nullptr);

// ---- moa.cu : the attention step of the mixture-of-attention-heads layer
bool moa_supported(const dsmoe_layer_desc& p, int n_head, int L);
// qa [Amax, H] bf16: the grouped rows' queries on entry, their attention outputs on return
dsmoe_status launch_moa_attention(const dsmoe_layer_desc& p, const MoaCore& c, void* qa, const int32_t* row_token,
                                  const int32_t* token_rows, const int32_t* offsets, int32_t* dev_status, cudaStream_t s);
// Whole-layer paths that need no grouping (all experts selected, or few tokens).  *done = false
// means "not taken": the caller continues with the grouped path.
// Whole layer for few tokens (T <= 128) in one cooperative launch, router included.
bool small_supported(const dsmoe_layer_desc& p);
dsmoe_status launch_layer_small(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                const void* packed, float* scores, uint64_t* mask, int32_t* k_t, int32_t* counts_out,
                                void* out, char* ws, const WsLayout& L, int32_t* dev_status, cudaStream_t s);
dsmoe_status launch_layer_umma(const dsmoe_layer_desc& p, const void* x, const void* packed, const float* scores,
                               const uint64_t* mask, const int32_t* k_t, int32_t* counts_out, void* out, char* ws,
                               const WsLayout& L, int32_t* dev_status, cudaStream_t s, bool* done);

// ---- training.cu / mlp_umma.cu : the training side (Eq. 2-6)
size_t mi_scratch_bytes();
dsmoe_status launch_mi_loss(const dsmoe_layer_desc& p, const float* scores, float* out3, float* grad, char* scratch,
                            cudaStream_t s);
dsmoe_status launch_dense_backward_plain(const dsmoe_layer_desc& p, const void* x, const void* W1, const void* W2,
                                         const float* scores, const uint64_t* mask, const void* dO, float* dS, void* dA,
                                         cudaStream_t s);
dsmoe_status launch_dense_backward(const dsmoe_layer_desc& p, const void* x, const void* W2, const void* packed,
                                   const float* scores, const uint64_t* mask, const void* dO, float* dS, void* dA,
                                   void* act, float* dot_part, int32_t* dev_status, cudaStream_t s);

}  // namespace dsmoe
