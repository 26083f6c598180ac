// C entry points of the dsmoe library: argument validation, workspace carving and the dispatch
// between the execution paths of one MoE layer call (Eq. 1).
#include "common.cuh"

namespace dsmoe {

dsmoe_status check_desc(const dsmoe_layer_desc* p) {
    if (!p) return DSMOE_ERR_INVALID_ARG;
    if (p->T < 0 || p->d <= 0 || p->H <= 0 || p->E <= 0) return DSMOE_ERR_INVALID_ARG;
    if (p->dtype != DSMOE_F32 && p->dtype != DSMOE_BF16) return DSMOE_ERR_INVALID_ARG;
    if (p->mode != DSMOE_SELECT_THRESHOLD && p->mode != DSMOE_SELECT_TOPK && p->mode != DSMOE_SELECT_ALL &&
        p->mode != DSMOE_SELECT_THRESHOLD_TOPK)
        return DSMOE_ERR_INVALID_ARG;
    if (p->mode == DSMOE_SELECT_TOPK && p->K < 1) return DSMOE_ERR_INVALID_ARG;
    if (p->min_k != 0 && p->min_k != 1) return DSMOE_ERR_INVALID_ARG;
    if (p->eps_normalized != 0 && p->eps_normalized != 1) return DSMOE_ERR_INVALID_ARG;
    if (p->out_fp32 != 0 && p->out_fp32 != 1) return DSMOE_ERR_INVALID_ARG;
    if (p->fuse_combine < 0 || p->fuse_combine > 2) return DSMOE_ERR_INVALID_ARG;
    if ((p->mode == DSMOE_SELECT_THRESHOLD || p->mode == DSMOE_SELECT_THRESHOLD_TOPK) && !(p->eps == p->eps))
        return DSMOE_ERR_INVALID_ARG;   // NaN
    if ((p->d & 7) || (p->H & 7)) return DSMOE_ERR_INVALID_ARG;
    if (p->E > kMaxExperts) return DSMOE_ERR_UNSUPPORTED;
    // every per-assignment index is an int32
    if ((double)p->T * p->E * (double)(p->d > p->H ? p->d : p->H) > 9.0e15) return DSMOE_ERR_UNSUPPORTED;
    if ((size_t)p->T * (size_t)p->E > 0x7fffffffull) return DSMOE_ERR_UNSUPPORTED;
    return DSMOE_OK;
}

WsLayout ws_layout(const dsmoe_layer_desc& p) {
    WsLayout L{};
    const size_t T = (size_t)p.T, E = (size_t)p.E, amax = amax_of(p), es = elem_size(p.dtype);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    L.scores = take(T * E * 4);
    L.mask = take(T * 8);
    L.k_t = take(T * 4);
    L.counts = take(kMaxExperts * 4);
    L.offsets = take((kMaxExperts + 1) * 4);
    L.chunk_prefix = take((size_t)ceil_div(p.T, kChunk) * E * 4);
    L.batch_k = take(256);               // Threshold-TopK: the batch's K
    L.sync = take(64);                   // grid-barrier counters of the small-T kernel
    L.tile_done = take((size_t)kMaxExperts * ceil_div(p.d, 256) * 4);   // grouped down-projection: finished tiles per (expert, column range)
    L.mi = take(mi_scratch_bytes());     // mutual-information loss: per-block partial sums
    L.row_token = take(amax * 4);
    L.row_gate = take(amax * 4);
    L.token_rows = take(T * (size_t)width_of(p) * 4);
    L.stage_total = off;
    const size_t big0 = off;
    // plain path: grouped copy of the tokens, fp32 hidden activations, expert outputs
    L.xp = take(amax * p.d * es);
    L.h_plain = take(amax * p.H * 4);
    L.yp = take(amax * p.d * es);
    L.total_plain = off;
    // tensor-core paths (bf16, packed weights); they start where the plain path's buffers start
    off = big0;
    size_t h_bytes = 0;
    if (umma_supported(p)) {
        h_bytes = amax * p.H * 2;                                   // grouped: [Amax, H]
        if (T * E * p.H * 2 > h_bytes) h_bytes = T * E * p.H * 2;       // dense forward and backward, small-T: [T, E*H]
    }
    L.h = take(h_bytes);
    // grouped: the tokens' fp32 running sums [T,d] (aggregation inside the down-projection), or the gate-weighted
    // expert outputs [Amax,d] in fp32 (separate aggregation)
    L.acc = take(!umma_supported(p) ? 0 : fuses_combine(p) ? T * p.d * 4 : amax * p.d * 4);
    // fp32 partial sums of the small-T path: (CTA, 2 column ranges, T, 256)
    L.partial = take(umma_supported(p) && p.T <= kSmallMaxT ? (size_t)kSmallMaxCtas * 2 * T * 256 * 4 : 0);
    L.router = take(router_umma_supported(p) ? router_umma_scratch(p) : 0);   // tensor-core router: split Wr, partial logits
    // dense backward: the experts' hidden activations go to `h` ([T,E*H]); per-column-tile partial dot products here
    L.bwd = take(umma_supported(p) ? T * E * ceil_div(p.H, 256) * 4 : 0);
    L.total_packed = off;
    L.total = L.total_plain > L.total_packed ? L.total_plain : L.total_packed;
    return L;
}

namespace {
DeviceState g_dev_state[kMaxDeviceSlots];
}

dsmoe_status device_state(DeviceState** out, int* device) {
    int dev = -1;
    DSMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDeviceSlots) return DSMOE_ERR_UNSUPPORTED;
    DeviceState& st = g_dev_state[dev];
    if (!st.sm_count) {
        int n = 0;
        DSMOE_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        if (n <= 0) return DSMOE_ERR_CUDA;
        st.sm_count = n;
    }
    *out = &st;
    if (device) *device = dev;
    return DSMOE_OK;
}

static const char* const kStatusText[] = {
    "ok", "invalid argument", "unsupported configuration", "workspace too small", "CUDA call failed",
    "bounded wait expired on the device"};

}  // namespace dsmoe

using namespace dsmoe;

extern "C" {

const char* dsmoe_status_string(dsmoe_status s) {
    return ((int)s >= 0 && (int)s <= 5) ? kStatusText[(int)s] : "unknown status";
}

dsmoe_status dsmoe_workspace_size(const dsmoe_layer_desc* desc, size_t* bytes) {
    DSMOE_TRY(check_desc(desc));
    if (!bytes) return DSMOE_ERR_INVALID_ARG;
    *bytes = ws_layout(*desc).total;
    return DSMOE_OK;
}

dsmoe_status dsmoe_workspace_size_packed(const dsmoe_layer_desc* desc, size_t* bytes) {
    DSMOE_TRY(check_desc(desc));
    if (!bytes) return DSMOE_ERR_INVALID_ARG;
    if (!umma_supported(*desc)) return DSMOE_ERR_UNSUPPORTED;
    *bytes = ws_layout(*desc).total_packed;
    return DSMOE_OK;
}

dsmoe_status dsmoe_workspace_size_stages(const dsmoe_layer_desc* desc, size_t* bytes) {
    DSMOE_TRY(check_desc(desc));
    if (!bytes) return DSMOE_ERR_INVALID_ARG;
    *bytes = ws_layout(*desc).stage_total;
    return DSMOE_OK;
}

dsmoe_status dsmoe_router(const dsmoe_layer_desc* desc, const void* x, const float* Wr, const float* br,
                          float* scores, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!x || !Wr || !scores || !aligned16(x) || !aligned16(Wr)) return DSMOE_ERR_INVALID_ARG;
    return launch_router(*desc, x, Wr, br, scores, nullptr, nullptr, (cudaStream_t)stream);
}

dsmoe_status dsmoe_select(const dsmoe_layer_desc* desc, const float* scores, uint64_t* mask, int32_t* k_t,
                          int32_t* counts, int32_t* offsets, void* workspace, size_t ws_bytes,
                          dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (!mask && desc->T > 0) return DSMOE_ERR_INVALID_ARG;
    if (!counts || !offsets || (!scores && desc->T > 0) || (!k_t && desc->T > 0)) return DSMOE_ERR_INVALID_ARG;
    const WsLayout L = ws_layout(*desc);
    if (!workspace || ws_bytes < L.stage_total) return DSMOE_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = (cudaStream_t)stream;
    DSMOE_TRY(launch_select(*desc, scores, mask, k_t, s, reinterpret_cast<int*>(ws + L.batch_k)));
    return launch_finalize(*desc, mask, counts, offsets, reinterpret_cast<int32_t*>(ws + L.chunk_prefix), nullptr, s);
}

dsmoe_status dsmoe_permute(const dsmoe_layer_desc* desc, const void* x, const float* scores, const uint64_t* mask,
                           const int32_t* offsets, int32_t* row_token, float* row_gate, int32_t* token_rows,
                           void* xp, void* workspace, size_t ws_bytes, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!x || !scores || !mask || !offsets || !row_token || !row_gate || !token_rows || !xp) return DSMOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(xp)) return DSMOE_ERR_INVALID_ARG;
    const WsLayout L = ws_layout(*desc);
    if (!workspace || ws_bytes < L.stage_total) return DSMOE_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = (cudaStream_t)stream;
    // recompute the per-chunk ranks from the mask (the caller's offsets are used as given)
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
    int32_t* offs_scratch = reinterpret_cast<int32_t*>(ws + L.offsets);
    int32_t* chunk_prefix = reinterpret_cast<int32_t*>(ws + L.chunk_prefix);
    DSMOE_TRY(launch_finalize(*desc, mask, counts, offs_scratch, chunk_prefix, nullptr, s));
    return launch_permute(*desc, x, scores, mask, offsets, chunk_prefix, row_token, row_gate, token_rows, xp, s);
}

dsmoe_status dsmoe_expert_mlp(const dsmoe_layer_desc* desc, const void* xp, const void* W1, const void* W2,
                              const void* packed, const int32_t* offsets, void* yp, void* workspace,
                              size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!xp || !offsets || !yp || !aligned16(xp) || !aligned16(yp)) return DSMOE_ERR_INVALID_ARG;
    if (packed && desc->dtype != DSMOE_BF16) return DSMOE_ERR_INVALID_ARG;
    if (!packed && (!W1 || !W2 || !aligned16(W1) || !aligned16(W2))) return DSMOE_ERR_INVALID_ARG;
    const WsLayout L = ws_layout(*desc);
    const bool fast = packed && umma_supported(*desc);
    if (!fast && (!W1 || !W2)) return DSMOE_ERR_UNSUPPORTED;   // packed weights given, but this shape needs the plain path
    if (!workspace || ws_bytes < (fast ? L.total_packed : L.total_plain)) return DSMOE_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = (cudaStream_t)stream;
    if (fast) return launch_mlp_umma(*desc, xp, packed, offsets, ws + L.h, yp, dev_status, s);
    return launch_mlp_generic(*desc, xp, W1, W2, offsets, reinterpret_cast<float*>(ws + L.h_plain), yp, s);
}

dsmoe_status dsmoe_combine(const dsmoe_layer_desc* desc, const void* yp, const float* row_gate,
                           const int32_t* token_rows, const int32_t* k_t, void* out, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!yp || !row_gate || !token_rows || !k_t || !out || !aligned16(yp) || !aligned16(out)) return DSMOE_ERR_INVALID_ARG;
    return launch_combine(*desc, yp, row_gate, token_rows, k_t, out, (cudaStream_t)stream);
}

dsmoe_status dsmoe_packed_size(const dsmoe_layer_desc* desc, size_t* bytes) {
    DSMOE_TRY(check_desc(desc));
    if (!bytes || desc->dtype != DSMOE_BF16) return DSMOE_ERR_INVALID_ARG;
    *bytes = (size_t)2 * desc->E * desc->H * desc->d * 2;
    return DSMOE_OK;
}

dsmoe_status dsmoe_pack_weights(const dsmoe_layer_desc* desc, const void* W1, const void* W2, void* packed,
                                dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->dtype != DSMOE_BF16 || !W1 || !W2 || !packed || !aligned16(packed)) return DSMOE_ERR_INVALID_ARG;
    if ((desc->d % 64) || (desc->H % 64)) return DSMOE_ERR_UNSUPPORTED;   // the packed layout is in blocks of 64
    return launch_pack(*desc, W1, W2, packed, (cudaStream_t)stream);
}

dsmoe_status dsmoe_layer_forward(const dsmoe_layer_desc* desc, const void* x, const float* Wr, const float* br,
                                 const void* W1, const void* W2, const void* packed, void* out,
                                 uint64_t* mask_out, int32_t* counts_out, void* workspace, size_t ws_bytes,
                                 int32_t* dev_status, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    const dsmoe_layer_desc& p = *desc;
    if (p.T == 0) return DSMOE_OK;
    if (!x || !Wr || !out || !aligned16(x) || !aligned16(Wr) || !aligned16(out)) return DSMOE_ERR_INVALID_ARG;
    if (packed && p.dtype != DSMOE_BF16) return DSMOE_ERR_INVALID_ARG;
    if (!packed && (!W1 || !W2 || !aligned16(W1) || !aligned16(W2))) return DSMOE_ERR_INVALID_ARG;
    const WsLayout L = ws_layout(p);
    const bool fast = packed && umma_supported(p);
    if (!fast && (!W1 || !W2)) return DSMOE_ERR_UNSUPPORTED;   // this shape needs the unpacked weights
    if (!workspace || ws_bytes < (fast ? L.total_packed : L.total_plain) || !aligned16(workspace)) return DSMOE_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = (cudaStream_t)stream;

    float* scores = reinterpret_cast<float*>(ws + L.scores);
    uint64_t* mask = mask_out ? mask_out : reinterpret_cast<uint64_t*>(ws + L.mask);
    int32_t* k_t = reinterpret_cast<int32_t*>(ws + L.k_t);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
    int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
    int32_t* chunk_prefix = reinterpret_cast<int32_t*>(ws + L.chunk_prefix);
    int32_t* row_token = reinterpret_cast<int32_t*>(ws + L.row_token);
    float* row_gate = reinterpret_cast<float*>(ws + L.row_gate);
    int32_t* token_rows = reinterpret_cast<int32_t*>(ws + L.token_rows);

    if (fast && small_supported(p))
        return launch_layer_small(p, x, Wr, br, packed, scores, mask, k_t, counts_out, out, ws, L, dev_status, s);

    // Threshold-TopK needs the whole batch's threshold counts before any token can be selected: the router runs
    // with the threshold rule, then the selection is redone with the batch's K
    dsmoe_layer_desc pr = p;
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) pr.mode = DSMOE_SELECT_THRESHOLD;
    // the tensor-core router leaves the per-chunk counts of its own selection behind (not Threshold-TopK's: that one
    // selects again)
    const bool counted = fast && router_umma_supported(p) && p.mode != DSMOE_SELECT_THRESHOLD_TOPK;
    if (fast && router_umma_supported(p))
        DSMOE_TRY(launch_router_umma(pr, x, Wr, br, scores, mask, k_t, ws + L.router, dev_status, s, counted ? chunk_prefix : nullptr));
    else
        DSMOE_TRY(launch_router(pr, x, Wr, br, scores, mask, k_t, s));
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK)
        DSMOE_TRY(launch_select(p, scores, mask, k_t, s, reinterpret_cast<int*>(ws + L.batch_k)));
    if (fast) {
        bool done = false;
        DSMOE_TRY(launch_layer_umma(p, x, packed, scores, mask, k_t, counts_out, out, ws, L, dev_status, s, &done));
        if (done) return DSMOE_OK;
    }

    // grouped path: duplicate tokens per selected expert, run the experts, aggregate
    if (fast && fuses_combine(p)) {
        // no grouped copy of the tokens (the up-projection gathers rows of x by row_token), no buffer of expert
        // outputs and no aggregation pass: the down-projection's epilogue adds each expert's gate-weighted output
        // to the token's fp32 sum, in ascending expert order, and writes the final rounding
        DSMOE_TRY(launch_group(p, scores, mask, counts, offsets, chunk_prefix, counts_out, row_token, row_gate, token_rows, s, out, counted));
        const CombineArgs cmb{row_token, row_gate, mask, reinterpret_cast<float*>(ws + L.acc),
                              reinterpret_cast<int*>(ws + L.tile_done), out};
        return launch_mlp_umma(p, nullptr, packed, offsets, ws + L.h, nullptr, dev_status, s, x, row_token, &cmb);
    }
    if (fast) {
        // the down-projection's epilogue multiplies by the gate and stores fp32 rows; the aggregation only adds
        DSMOE_TRY(launch_group(p, scores, mask, counts, offsets, chunk_prefix, counts_out, row_token, row_gate, token_rows, s, nullptr, counted));
        const CombineArgs gated{row_token, row_gate, nullptr, nullptr, nullptr, nullptr};
        DSMOE_TRY(launch_mlp_umma(p, nullptr, packed, offsets, ws + L.h, ws + L.acc, dev_status, s, x, row_token, &gated));
        return launch_combine(p, ws + L.acc, nullptr, token_rows, k_t, out, s, true);
    }
    DSMOE_TRY(launch_finalize(p, mask, counts, offsets, chunk_prefix, counts_out, s));
    DSMOE_TRY(launch_permute(p, x, scores, mask, offsets, chunk_prefix, row_token, row_gate, token_rows, ws + L.xp, s));
    DSMOE_TRY(launch_mlp_generic(p, ws + L.xp, W1, W2, offsets, reinterpret_cast<float*>(ws + L.h_plain), ws + L.yp, s));
    return launch_combine(p, ws + L.yp, row_gate, token_rows, k_t, out, s);
}

dsmoe_status dsmoe_layer_forward_host_async(const dsmoe_layer_desc* desc, const void* x_host, void* x_dev,
                                            const float* Wr, const float* br, const void* W1, const void* W2,
                                            const void* packed, void* out_dev, void* out_host, void* workspace,
                                            size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!x_host || !x_dev || !out_dev || !out_host) return DSMOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t n = (size_t)desc->T * desc->d;
    const size_t out_es = desc->out_fp32 ? 4 : elem_size(desc->dtype);
    DSMOE_CUDA_TRY(cudaMemcpyAsync(x_dev, x_host, n * elem_size(desc->dtype), cudaMemcpyHostToDevice, s));
    DSMOE_TRY(dsmoe_layer_forward(desc, x_dev, Wr, br, W1, W2, packed, out_dev, nullptr, nullptr, workspace, ws_bytes,
                                  dev_status, stream));
    DSMOE_CUDA_TRY(cudaMemcpyAsync(out_host, out_dev, n * out_es, cudaMemcpyDeviceToHost, s));
    return DSMOE_OK;
}

dsmoe_status dsmoe_layer_forward_host(const dsmoe_layer_desc* desc, const void* x_host, void* x_dev,
                                      const float* Wr, const float* br, const void* W1, const void* W2,
                                      const void* packed, void* out_dev, void* out_host, void* workspace,
                                      size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream) {
    DSMOE_TRY(dsmoe_layer_forward_host_async(desc, x_host, x_dev, Wr, br, W1, W2, packed, out_dev, out_host, workspace,
                                             ws_bytes, dev_status, stream));
    if (desc->T == 0) return DSMOE_OK;
    DSMOE_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return DSMOE_OK;
}

dsmoe_status dsmoe_stats(const dsmoe_layer_desc* desc, const float* scores, const uint64_t* mask,
                         dsmoe_selection_stats* stats, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (!stats || (desc->T > 0 && (!scores || !mask))) return DSMOE_ERR_INVALID_ARG;
    return launch_stats(*desc, scores, mask, stats, (cudaStream_t)stream);
}

dsmoe_status dsmoe_mi_loss(const dsmoe_layer_desc* desc, const float* scores, float* loss3, float* grad,
                           void* workspace, size_t ws_bytes, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0 || !scores || !loss3) return DSMOE_ERR_INVALID_ARG;
    const WsLayout L = ws_layout(*desc);
    if (!workspace || ws_bytes < L.stage_total) return DSMOE_ERR_WORKSPACE;
    return launch_mi_loss(*desc, scores, loss3, grad, static_cast<char*>(workspace) + L.mi, (cudaStream_t)stream);
}

dsmoe_status dsmoe_dense_backward(const dsmoe_layer_desc* desc, const void* x, const void* W1, const void* W2,
                                  const void* packed, const float* scores, const uint64_t* mask, const void* dO,
                                  float* dS, void* dA, void* workspace, size_t ws_bytes, int32_t* dev_status,
                                  dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (desc->T == 0) return DSMOE_OK;
    if (!x || !W2 || !scores || !dO || !dS || !dA) return DSMOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W2) || !aligned16(dO) || !aligned16(dA)) return DSMOE_ERR_INVALID_ARG;
    if (packed && desc->dtype != DSMOE_BF16) return DSMOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (packed && umma_supported(*desc)) {
        const WsLayout L = ws_layout(*desc);
        if (!workspace || ws_bytes < L.total_packed || !aligned16(workspace)) return DSMOE_ERR_WORKSPACE;
        char* ws = static_cast<char*>(workspace);
        return launch_dense_backward(*desc, x, W2, packed, scores, mask, dO, dS, dA, ws + L.h,
                                     reinterpret_cast<float*>(ws + L.bwd), dev_status, s);
    }
    if (!W1 || !aligned16(W1)) return packed ? DSMOE_ERR_UNSUPPORTED : DSMOE_ERR_INVALID_ARG;
    return launch_dense_backward_plain(*desc, x, W1, W2, scores, mask, dO, dS, dA, s);
}

dsmoe_status dsmoe_moa_forward(const dsmoe_layer_desc* desc, const dsmoe_moa_args* args, const void* x, const float* Wr,
                               const float* br, const void* packed, void* out, uint64_t* mask_out, int32_t* counts_out,
                               void* workspace, size_t ws_bytes, int32_t* dev_status, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    const dsmoe_layer_desc& p = *desc;
    if (p.T == 0) return DSMOE_OK;
    if (!args || !x || !Wr || !out || !packed || !args->Kc || !args->Vc || !args->pos) return DSMOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(Wr) || !aligned16(out) || !aligned16(packed) || !aligned16(args->Kc) || !aligned16(args->Vc))
        return DSMOE_ERR_INVALID_ARG;
    if (args->n_seq <= 0 || args->L <= 0) return DSMOE_ERR_INVALID_ARG;
    if (p.dtype != DSMOE_BF16 || !moa_supported(p, args->n_head, args->L)) return DSMOE_ERR_UNSUPPORTED;
    const WsLayout L = ws_layout(p);
    if (!workspace || ws_bytes < L.total_packed || !aligned16(workspace)) return DSMOE_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = (cudaStream_t)stream;
    float* scores = reinterpret_cast<float*>(ws + L.scores);
    uint64_t* mask = mask_out ? mask_out : reinterpret_cast<uint64_t*>(ws + L.mask);
    int32_t* k_t = reinterpret_cast<int32_t*>(ws + L.k_t);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
    int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
    int32_t* chunk_prefix = reinterpret_cast<int32_t*>(ws + L.chunk_prefix);
    int32_t* row_token = reinterpret_cast<int32_t*>(ws + L.row_token);
    float* row_gate = reinterpret_cast<float*>(ws + L.row_gate);
    int32_t* token_rows = reinterpret_cast<int32_t*>(ws + L.token_rows);
    const MoaCore core{args->n_head, args->n_seq, args->L, args->scale, args->Kc, args->Vc, args->tok_seq, args->pos, token_rows};

    // router, selection and grouping as in dsmoe_layer_forward's grouped path (also when every expert is selected)
    dsmoe_layer_desc pr = p;
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) pr.mode = DSMOE_SELECT_THRESHOLD;
    // the tensor-core router leaves the per-chunk counts of its own selection behind (not Threshold-TopK's: that one
    // selects again)
    const bool counted = router_umma_supported(p) && p.mode != DSMOE_SELECT_THRESHOLD_TOPK;
    if (router_umma_supported(p))
        DSMOE_TRY(launch_router_umma(pr, x, Wr, br, scores, mask, k_t, ws + L.router, dev_status, s, counted ? chunk_prefix : nullptr));
    else
        DSMOE_TRY(launch_router(pr, x, Wr, br, scores, mask, k_t, s));
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK)
        DSMOE_TRY(launch_select(p, scores, mask, k_t, s, reinterpret_cast<int*>(ws + L.batch_k)));
    if (fuses_combine(p)) {
        DSMOE_TRY(launch_group(p, scores, mask, counts, offsets, chunk_prefix, counts_out, row_token, row_gate, token_rows, s, out, counted));
        const CombineArgs cmb{row_token, row_gate, mask, reinterpret_cast<float*>(ws + L.acc),
                              reinterpret_cast<int*>(ws + L.tile_done), out};
        return launch_mlp_umma(p, nullptr, packed, offsets, ws + L.h, nullptr, dev_status, s, x, row_token, &cmb, &core);
    }
    DSMOE_TRY(launch_group(p, scores, mask, counts, offsets, chunk_prefix, counts_out, row_token, row_gate, token_rows, s, nullptr, counted));
    const CombineArgs gated{row_token, row_gate, nullptr, nullptr, nullptr, nullptr};
    DSMOE_TRY(launch_mlp_umma(p, nullptr, packed, offsets, ws + L.h, ws + L.acc, dev_status, s, x, row_token, &gated, &core));
    return launch_combine(p, ws + L.acc, nullptr, token_rows, k_t, out, s, true);
}

dsmoe_status dsmoe_timing_enable(int n_pairs) {
    if (n_pairs < 0 || n_pairs > (1 << 20)) return DSMOE_ERR_INVALID_ARG;
    return timing_enable(n_pairs);
}

dsmoe_status dsmoe_timing_read(float* ms, int n_max, int* n) {
    if (!ms || !n || n_max < 0) return DSMOE_ERR_INVALID_ARG;
    return timing_read(ms, n_max, n);
}

}  // extern "C"
