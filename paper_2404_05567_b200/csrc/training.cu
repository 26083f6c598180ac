// Training side of the layer: the mutual-information loss of the router (Eq. 4-6) and a plain fp32-FMA version of
// the gradients of dense training (Eq. 2, Eq. 3) for fp32 layers and shapes the tensor-core path does not take.
#include "common.cuh"

namespace dsmoe {

namespace {

constexpr int kMiBlocks = 296;        // upper bound on the first stage's grid (sizes its partial-sum buffer)

// Stage 1: block b adds its tokens' scores per expert and their conditional entropies, in double, in a fixed order
// (warp w of the block takes tokens w, w + 8, ...; lanes hold experts lane and lane + 32; the warps' sums meet in shared
// memory and are added in warp order).  part[b][0..E) = sum_t S[t,e], part[b][64] = sum_t H(e|X_t).
__global__ void __launch_bounds__(256) mi_partial_kernel(const float* __restrict__ S, double* __restrict__ part, int T, int E) {
    __shared__ double red[8][kMaxExperts + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int per = (T + gridDim.x - 1) / gridDim.x;
    const int t0 = blockIdx.x * per, t1 = min(T, t0 + per);
    double p_lo = 0.0, p_hi = 0.0, h = 0.0;
    for (int t = t0 + warp; t < t1; t += 8) {
        const float s_lo = lane < E ? S[(size_t)t * E + lane] : 0.f;
        const float s_hi = lane + 32 < E ? S[(size_t)t * E + lane + 32] : 0.f;
        p_lo += (double)s_lo;
        p_hi += (double)s_hi;
        double hv = 0.0;
        if (s_lo > 0.f) hv -= (double)s_lo * log((double)s_lo);
        if (s_hi > 0.f) hv -= (double)s_hi * log((double)s_hi);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) hv += __shfl_xor_sync(0xffffffffu, hv, o);
        h += hv;
    }
    red[warp][lane] = p_lo;
    red[warp][lane + 32] = p_hi;
    if (lane == 0) red[warp][kMaxExperts] = h;
    __syncthreads();
    if (threadIdx.x <= kMaxExperts) {
        double v = 0.0;
        for (int w = 0; w < 8; ++w) v += red[w][threadIdx.x];
        part[(size_t)blockIdx.x * (kMaxExperts + 1) + threadIdx.x] = v;
    }
}

// Stage 2: one block.  p(e) = mean score, H(e), mean H(e|X), L_MI = -H(e) + mean H(e|X); p(e) is left in `pe`.
__global__ void __launch_bounds__(64) mi_finish_kernel(const double* __restrict__ part, int nblocks, int T, int E,
                                                       float* __restrict__ out3, double* __restrict__ pe) {
    __shared__ double term[kMaxExperts];
    const int e = threadIdx.x;
    double v = 0.0;
    if (e < E) {
        for (int b = 0; b < nblocks; ++b) v += part[(size_t)b * (kMaxExperts + 1) + e];
        v /= (double)T;
        pe[e] = v;
    }
    term[e] = (e < E && v > 0.0) ? -v * log(v) : 0.0;
    __syncthreads();
    if (e == 0) {
        double he = 0.0, hc = 0.0;
        for (int i = 0; i < E; ++i) he += term[i];
        for (int b = 0; b < nblocks; ++b) hc += part[(size_t)b * (kMaxExperts + 1) + kMaxExperts];
        hc /= (double)T;
        out3[0] = (float)(-he + hc);
        out3[1] = (float)he;
        out3[2] = (float)hc;
    }
}

// dL_MI/dS[t,e] = (log p(e) - log S[t,e]) / T   (0 where the score is 0)
__global__ void __launch_bounds__(256) mi_grad_kernel(const float* __restrict__ S, const double* __restrict__ pe,
                                                      float* __restrict__ grad, long long n, int T, int E) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const float s = S[i];
    grad[i] = s > 0.f ? (float)((log(pe[i % E]) - log((double)s)) / (double)T) : 0.f;
}

__device__ __forceinline__ float ldv(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ldv(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stv(float* p, float v) { *p = v; }
__device__ __forceinline__ void stv(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// One block per (token, expert): every thread takes hidden units k = tid, tid + 256, ...; for each it forms the hidden
// activation a_k = GeLU(x.W1[e][:,k]) and G_k = dO.W2[e][k,:], writes dA = S * G_k and adds a_k * G_k to the block's
// dot product, which is <e_e(x), dO>.
template <typename XT>
__global__ void __launch_bounds__(256) dense_backward_plain_kernel(const XT* __restrict__ x, const XT* __restrict__ W1,
                                                                   const XT* __restrict__ W2, const float* __restrict__ S,
                                                                   const uint64_t* __restrict__ mask, const XT* __restrict__ dO,
                                                                   float* __restrict__ dS, XT* __restrict__ dA, int d, int H, int E) {
    __shared__ float red[8];
    const int t = blockIdx.x / E, e = blockIdx.x % E;
    const bool active = !mask || ((mask[t] >> e) & 1ull);
    const float gate = active ? S[(size_t)t * E + e] : 0.f;
    const XT* xr = x + (size_t)t * d;
    const XT* gr = dO + (size_t)t * d;
    float dot = 0.f;
    for (int k = threadIdx.x; k < H; k += 256) {
        float pre = 0.f, G = 0.f;
        if (active) {
            const XT* w1 = W1 + (size_t)e * d * H + k;
            const XT* w2 = W2 + ((size_t)e * H + k) * d;
            for (int c = 0; c < d; ++c) {
                pre = fmaf(ldv(xr + c), ldv(w1 + (size_t)c * H), pre);
                G = fmaf(ldv(gr + c), ldv(w2 + c), G);
            }
            const float a = 0.5f * pre * (1.f + erff(pre * 0.70710678118654752440f));
            dot = fmaf(a, G, dot);
        }
        stv(dA + ((size_t)t * E + e) * H + k, gate * G);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = dot;
    __syncthreads();
    if (threadIdx.x == 0) {
        float v = 0.f;
        for (int w = 0; w < 8; ++w) v += red[w];
        dS[(size_t)t * E + e] = v;
    }
}

}  // namespace

size_t mi_scratch_bytes() { return (size_t)kMiBlocks * (kMaxExperts + 1) * sizeof(double) + kMaxExperts * sizeof(double); }

dsmoe_status launch_mi_loss(const dsmoe_layer_desc& p, const float* scores, float* out3, float* grad, char* scratch,
                            cudaStream_t s) {
    double* part = reinterpret_cast<double*>(scratch);
    double* pe = part + (size_t)kMiBlocks * (kMaxExperts + 1);
    const int nblocks = ceil_div(p.T, 64) < kMiBlocks ? ceil_div(p.T, 64) : kMiBlocks;
    mi_partial_kernel<<<nblocks, 256, 0, s>>>(scores, part, p.T, p.E);
    DSMOE_CUDA_TRY(cudaGetLastError());
    mi_finish_kernel<<<1, 64, 0, s>>>(part, nblocks, p.T, p.E, out3, pe);
    DSMOE_CUDA_TRY(cudaGetLastError());
    if (grad) {
        const long long n = (long long)p.T * p.E;
        mi_grad_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(scores, pe, grad, n, p.T, p.E);
        DSMOE_CUDA_TRY(cudaGetLastError());
    }
    return DSMOE_OK;
}

dsmoe_status launch_dense_backward_plain(const dsmoe_layer_desc& p, const void* x, const void* W1, const void* W2,
                                         const float* scores, const uint64_t* mask, const void* dO, float* dS, void* dA,
                                         cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    const unsigned grid = (unsigned)((size_t)p.T * p.E);
    if (p.dtype == DSMOE_BF16)
        dense_backward_plain_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(
            static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(W1), static_cast<const __nv_bfloat16*>(W2),
            scores, mask, static_cast<const __nv_bfloat16*>(dO), dS, static_cast<__nv_bfloat16*>(dA), p.d, p.H, p.E);
    else
        dense_backward_plain_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(x), static_cast<const float*>(W1),
                                                                static_cast<const float*>(W2), scores, mask,
                                                                static_cast<const float*>(dO), dS, static_cast<float*>(dA),
                                                                p.d, p.H, p.E);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace dsmoe
