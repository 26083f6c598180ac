// Device-side pieces of the router that more than one kernel uses: the per-token softmax over all
// experts (Eq. 1) and the selection rules ("Sparse Inference" paragraph; threshold on the normalised
// probability per the Results-section footnote), one warp per token.
#pragma once

#include "common.cuh"

namespace dsmoe {

struct SelParams {
    int E, mode;
    float eps;
    int eps_normalized, K, min_k;
    const int* K_dev;    // when set, the K of the top-K rule is read from here (Threshold-TopK: K comes from the batch)
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// Selection for one token held by a full warp.  s_lo / s_hi: fp32 scores of experts lane and
// lane + 32.  All comparisons are fp32 and exact, so equal scores give equal masks on any machine.
__device__ __forceinline__ uint64_t select_warp(float s_lo, float s_hi, const SelParams& q, int lane) {
    const bool v_lo = lane < q.E, v_hi = lane + 32 < q.E;
    bool sel_lo, sel_hi;
    if (q.mode == DSMOE_SELECT_THRESHOLD) {
        // "exceeds a threshold": strict >.  Normalised probability = S * N, one fp32 multiply.
        const float a_lo = q.eps_normalized ? __fmul_rn(s_lo, (float)q.E) : s_lo;
        const float a_hi = q.eps_normalized ? __fmul_rn(s_hi, (float)q.E) : s_hi;
        sel_lo = v_lo && a_lo > q.eps;
        sel_hi = v_hi && a_hi > q.eps;
    } else if (q.mode == DSMOE_SELECT_TOPK) {
        // rank = number of experts that beat this one (higher score, or equal score and lower index)
        const int K = q.K_dev ? *q.K_dev : q.K;
        int better_lo = 0, better_hi = 0;
        if (q.E <= 32) {                 // one expert per lane: half the comparisons
            for (int j = 0; j < q.E; ++j) {
                const float o = __shfl_sync(0xffffffffu, s_lo, j);
                better_lo += (o > s_lo) || (o == s_lo && j < lane);
            }
        } else {
            for (int j = 0; j < q.E; ++j) {
                const float o = j < 32 ? __shfl_sync(0xffffffffu, s_lo, j) : __shfl_sync(0xffffffffu, s_hi, j - 32);
                better_lo += (o > s_lo) || (o == s_lo && j < lane);
                better_hi += (o > s_hi) || (o == s_hi && j < lane + 32);
            }
        }
        sel_lo = v_lo && better_lo < K;
        sel_hi = v_hi && better_hi < K;
    } else {
        sel_lo = v_lo;
        sel_hi = v_hi;
    }
    uint64_t m = (uint64_t)__ballot_sync(0xffffffffu, sel_lo) | ((uint64_t)__ballot_sync(0xffffffffu, sel_hi) << 32);
    if (m == 0 && q.min_k == 1) {
        float best = v_lo ? s_lo : -INFINITY;
        int idx = lane;
        if (v_hi && s_hi > best) {
            best = s_hi;
            idx = lane + 32;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (ob > best || (ob == best && oi < idx)) {
                best = ob;
                idx = oi;
            }
        }
        m = (uint64_t)1 << idx;
    }
    return m;
}

// Softmax over all E experts of one token (row maximum subtracted), logits and scores of experts lane and
// lane + 32 held by a full warp.
__device__ __forceinline__ void softmax_warp(float l_lo, float l_hi, int E, int lane, float& s_lo, float& s_hi) {
    const bool v_lo = lane < E, v_hi = lane + 32 < E;
    const float mx = warp_max(fmaxf(v_lo ? l_lo : -INFINITY, v_hi ? l_hi : -INFINITY));
    const float p_lo = v_lo ? expf(l_lo - mx) : 0.f;
    const float p_hi = v_hi ? expf(l_hi - mx) : 0.f;
    const float den = warp_sum(p_lo + p_hi);
    s_lo = __fdiv_rn(p_lo, den);
    s_hi = __fdiv_rn(p_hi, den);
}

// Softmax, then selection; the warp writes scores[t,:], mask[t], k_t[t] (each optional) and returns the selection word
// (0 where neither mask nor k_t is asked for).
__device__ __forceinline__ uint64_t softmax_select_store(float l_lo, float l_hi, int t, const SelParams& q, int lane,
                                                         float* __restrict__ scores, uint64_t* __restrict__ mask,
                                                         int32_t* __restrict__ k_t) {
    const bool v_lo = lane < q.E, v_hi = lane + 32 < q.E;
    float s_lo, s_hi;
    softmax_warp(l_lo, l_hi, q.E, lane, s_lo, s_hi);
    if (scores) {
        if (v_lo) scores[(size_t)t * q.E + lane] = s_lo;
        if (v_hi) scores[(size_t)t * q.E + lane + 32] = s_hi;
    }
    uint64_t m = 0;
    if (mask || k_t) {
        m = select_warp(s_lo, s_hi, q, lane);
        if (lane == 0) {
            if (mask) mask[t] = m;
            if (k_t) k_t[t] = __popcll(m);
        }
    }
    return m;
}

}  // namespace dsmoe
