// Plain fp32-FMA grouped GEMMs for the expert MLPs (Eq. 1's e(X) = GeLU(X.W1).W2): the path for fp32
// layers and for bf16 layers whose weights have not been packed for the tensor-core kernels.
// Rows are grouped by expert (offsets[e] .. offsets[e+1]); a block computes one 64x64 output tile of
// one expert's segment.
#include "common.cuh"

namespace dsmoe {

__device__ __forceinline__ float ld_f32(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_f32(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f)); }

// C[r, n] = act( sum_k A[r, k] * B[e, k, n] ),  r in segment e.  A [rows,K], B [E,K,N], C [rows,N].
template <typename AT, typename BT, typename OT, bool GELU>
__global__ void __launch_bounds__(256) grouped_gemm_fma_kernel(const AT* __restrict__ A, const BT* __restrict__ B,
                                                               OT* __restrict__ C, const int32_t* __restrict__ offsets,
                                                               int E, int K, int N, int64_t amax) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN];
    // which expert segment and which row tile inside it
    int tile = blockIdx.x, e = 0, seg0 = 0, seg1 = 0;
    for (; e < E; ++e) {
        seg0 = offsets[e];
        seg1 = offsets[e + 1];
        const int tiles = (seg1 - seg0 + BM - 1) / BM;
        if (tile < tiles) break;
        tile -= tiles;
    }
    if (e == E || seg0 < 0 || seg1 > amax) return;
    const int r0 = seg0 + tile * BM, n0 = blockIdx.y * BN;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const BT* Be = B + (size_t)e * K * N;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int idx = tid; idx < BM * BK; idx += 256) {
            const int m = idx / BK, kk = idx % BK;
            const int r = r0 + m, k = k0 + kk;
            As[kk][m] = (r < seg1 && k < K) ? ld_f32(A + (size_t)r * K + k) : 0.f;
        }
        for (int idx = tid; idx < BK * BN; idx += 256) {
            const int kk = idx / BN, n = idx % BN;
            const int k = k0 + kk;
            Bs[kk][n] = (k < K && n0 + n < N) ? ld_f32(Be + (size_t)k * N + n0 + n) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty * 4 + i;
        if (r >= seg1) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx + 16 * j;
            if (n < N) st_out(C + (size_t)r * N + n, GELU ? gelu_erf(acc[i][j]) : acc[i][j]);
        }
    }
}

template <typename XT>
static dsmoe_status run(const dsmoe_layer_desc& p, const XT* xp, const XT* W1, const XT* W2, const int32_t* offsets,
                        float* h, XT* yp, cudaStream_t s) {
    const size_t amax = amax_of(p);
    const unsigned gx = (unsigned)(amax / 64 + p.E + 1);
    grouped_gemm_fma_kernel<XT, XT, float, true>
        <<<dim3(gx, ceil_div(p.H, 64)), 256, 0, s>>>(xp, W1, h, offsets, p.E, p.d, p.H, (int64_t)amax);
    DSMOE_CUDA_TRY(cudaGetLastError());
    grouped_gemm_fma_kernel<float, XT, XT, false>
        <<<dim3(gx, ceil_div(p.d, 64)), 256, 0, s>>>(h, W2, yp, offsets, p.E, p.H, p.d, (int64_t)amax);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_mlp_generic(const dsmoe_layer_desc& p, const void* xp, const void* W1, const void* W2,
                                const int32_t* offsets, float* h, void* yp, cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    if (p.dtype == DSMOE_BF16)
        return run(p, static_cast<const __nv_bfloat16*>(xp), static_cast<const __nv_bfloat16*>(W1),
                   static_cast<const __nv_bfloat16*>(W2), offsets, h, static_cast<__nv_bfloat16*>(yp), s);
    return run(p, static_cast<const float*>(xp), static_cast<const float*>(W1), static_cast<const float*>(W2), offsets,
               h, static_cast<float*>(yp), s);
}

}  // namespace dsmoe
