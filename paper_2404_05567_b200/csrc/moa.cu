// Mixture-of-attention-heads layer (Eq. 7-8): the attention step between the two grouped projections.
//
// The layer is the feed-forward layer's pipeline with another middle: router, selection and grouping as there; the
// "up-projection" is the experts' query projection (no activation), the "down-projection" their output projection
// with the router-weighted sum of Eq. 8; in between every grouped row -- one (token, expert) pair, n_head query
// vectors of d_head -- attends to the keys and values of its token's sequence, head j to key/value head j
// (the keys and values are shared by all experts).  This file holds that middle step.
#include "common.cuh"

namespace dsmoe {

namespace {

constexpr int kMoaWarps = 4;

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// One warp per (grouped row, head).  Pass 1: the lanes share out the visible keys, each key's logit is a full dot
// product of the query (fp32, in shared memory) with the key's row (read in 16-byte pieces); logits go to shared
// memory.  Then max, exponentials and their sum.  Pass 2: the lanes share out the d_head dimensions (lane l owns
// l, l + 32, ...) and walk the keys, so a value row is read by the whole warp at once.  The result replaces the
// query in place (the warp has read all of it before it writes).
template <int DPL>   // d_head / 32
__global__ void __launch_bounds__(32 * kMoaWarps)
moa_attention_kernel(__nv_bfloat16* __restrict__ qa, const int32_t* __restrict__ row_token, const int32_t* __restrict__ offsets,
                     int E, int n_head, int H, int T, const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                     const int32_t* __restrict__ tok_seq, const int32_t* __restrict__ pos, int n_seq, int L, float scale,
                     int* __restrict__ dev_status) {
    constexpr int DH = 32 * DPL;
    extern __shared__ float moa_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* qs = moa_smem + warp * (DH + ((L + 3) & ~3));     // the query, then the logits / probabilities
    float* ws = qs + DH;
    const long long A = offsets[E];
    const long long pair = (long long)blockIdx.x * kMoaWarps + warp;
    if (pair >= A * n_head) return;
    const long long r = pair / n_head;
    const int j = (int)(pair % n_head);
    int t = row_token[r];
    bool bad = t < 0 || t >= T;
    t = min(max(t, 0), T - 1);
    int sq = tok_seq ? tok_seq[t] : 0, last = pos[t];
    bad = bad || sq < 0 || sq >= n_seq || last < 0 || last >= L;
    if (bad) {                                        // report, and stay inside the cache
        if (lane == 0) *dev_status = DSMOE_ERR_INVALID_ARG;
        sq = min(max(sq, 0), n_seq - 1);
        last = min(max(last, 0), L - 1);
    }
    __nv_bfloat16* qrow = qa + r * H + j * DH;
#pragma unroll
    for (int i = 0; i < DPL; ++i) qs[lane + 32 * i] = __bfloat162float(qrow[lane + 32 * i]);
    __syncwarp();
    const __nv_bfloat16* Kh = Kc + ((size_t)(sq * n_head + j) * L) * DH;
    const __nv_bfloat16* Vh = Vc + ((size_t)(sq * n_head + j) * L) * DH;
    float mx = -INFINITY;
    for (int k = lane; k <= last; k += 32) {
        const uint4* kr = reinterpret_cast<const uint4*>(Kh + (size_t)k * DH);
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
            const uint4 u = __ldg(kr + c);
            const float4 q0 = *reinterpret_cast<const float4*>(qs + 8 * c), q1 = *reinterpret_cast<const float4*>(qs + 8 * c + 4);
            dot = fmaf(q0.x, bf16_lo(u.x), dot);
            dot = fmaf(q0.y, bf16_hi(u.x), dot);
            dot = fmaf(q0.z, bf16_lo(u.y), dot);
            dot = fmaf(q0.w, bf16_hi(u.y), dot);
            dot = fmaf(q1.x, bf16_lo(u.z), dot);
            dot = fmaf(q1.y, bf16_hi(u.z), dot);
            dot = fmaf(q1.z, bf16_lo(u.w), dot);
            dot = fmaf(q1.w, bf16_hi(u.w), dot);
        }
        dot *= scale;
        ws[k] = dot;
        mx = fmaxf(mx, dot);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float den = 0.f;
    for (int k = lane; k <= last; k += 32) {
        const float p = expf(ws[k] - mx);
        ws[k] = p;
        den += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    __syncwarp();
    float acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
    for (int k = 0; k <= last; ++k) {
        const float p = ws[k];
        const __nv_bfloat16* vr = Vh + (size_t)k * DH + lane;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] = fmaf(p, __bfloat162float(vr[32 * i]), acc[i]);
    }
    const float inv = 1.f / den;
#pragma unroll
    for (int i = 0; i < DPL; ++i) qrow[lane + 32 * i] = __float2bfloat16_rn(acc[i] * inv);
}

}  // namespace

bool moa_supported(const dsmoe_layer_desc& p, int n_head, int L) {
    if (!umma_supported(p) || n_head <= 0 || p.H % n_head) return false;
    const int dh = p.H / n_head;
    return dh % 32 == 0 && dh <= 256 && L > 0 && (size_t)(dh + L + 3) * 4 * kMoaWarps <= 200 * 1024;
}

dsmoe_status launch_moa_attention(const dsmoe_layer_desc& p, const MoaCore& c, void* qa, const int32_t* row_token,
                                  const int32_t* offsets, int32_t* dev_status, cudaStream_t s) {
    const int dh = p.H / c.n_head;
    int warps = kMoaWarps;
    const size_t per_warp = (size_t)(dh + ((c.L + 3) & ~3)) * 4;
    const size_t smem = per_warp * warps;
    if (smem > 200 * 1024) return DSMOE_ERR_UNSUPPORTED;
    const long long pairs = (long long)amax_of(p) * c.n_head;
    const unsigned grid = (unsigned)((pairs + warps - 1) / warps);
    auto* q = static_cast<__nv_bfloat16*>(qa);
    auto* K = static_cast<const __nv_bfloat16*>(c.Kc);
    auto* V = static_cast<const __nv_bfloat16*>(c.Vc);
#define MOA_LAUNCH(DPL)                                                                                                   \
    do {                                                                                                                  \
        if (smem > 48 * 1024)                                                                                             \
            DSMOE_CUDA_TRY(cudaFuncSetAttribute(moa_attention_kernel<DPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                                (int)smem));                                                              \
        moa_attention_kernel<DPL><<<grid, 32 * kMoaWarps, smem, s>>>(q, row_token, offsets, p.E, c.n_head, p.H, p.T, K, V, \
                                                                     c.tok_seq, c.pos, c.n_seq, c.L, c.scale, dev_status); \
    } while (0)
    switch (dh / 32) {
        case 1: MOA_LAUNCH(1); break;
        case 2: MOA_LAUNCH(2); break;
        case 3: MOA_LAUNCH(3); break;
        case 4: MOA_LAUNCH(4); break;
        case 5: MOA_LAUNCH(5); break;
        case 6: MOA_LAUNCH(6); break;
        case 7: MOA_LAUNCH(7); break;
        case 8: MOA_LAUNCH(8); break;
        default: return DSMOE_ERR_UNSUPPORTED;
    }
#undef MOA_LAUNCH
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace dsmoe
