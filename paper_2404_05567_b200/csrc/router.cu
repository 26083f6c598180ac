// Router scores (Eq. 1: S = softmax(h(X)), h linear), expert selection ("Sparse Inference"
// paragraph; threshold on the normalised probability per the Results-section footnote) and the
// per-expert counts / offsets that the grouping step needs.
//
// One warp owns one token from the logits onward: lane e holds expert e (and e+32 when E > 32), so
// the softmax and every selection rule are warp shuffles and ballots, and the selected set of a
// token is one 64-bit ballot word.
#include "common.cuh"
#include "router_device.cuh"

namespace dsmoe {

static SelParams sel_params(const dsmoe_layer_desc& p) {
    return SelParams{p.E, p.mode, p.eps, p.eps_normalized, p.K, p.min_k};
}

// Small T (decode): one block per token, the reduction over d split across all 256 threads.
template <typename XT, int EP>
__global__ void __launch_bounds__(256) router_small_kernel(const XT* __restrict__ x, const float* __restrict__ Wr,
                                                           const float* __restrict__ br, float* __restrict__ scores,
                                                           uint64_t* __restrict__ mask, int32_t* __restrict__ k_t,
                                                           int d, SelParams q) {
    __shared__ float red[8][EP];
    const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int E = q.E;
    float acc[EP];
#pragma unroll
    for (int e = 0; e < EP; ++e) acc[e] = 0.f;
    const XT* xr = x + (size_t)t * d;
    if ((E & 3) == 0) {
        for (int k = tid; k < d; k += 256) {
            const float xv = to_f32(xr[k]);
            const float4* w = reinterpret_cast<const float4*>(Wr + (size_t)k * E);
#pragma unroll
            for (int e4 = 0; e4 < EP / 4; ++e4) {
                if (e4 * 4 < E) {
                    const float4 wv = __ldg(w + e4);
                    acc[e4 * 4 + 0] = fmaf(xv, wv.x, acc[e4 * 4 + 0]);
                    acc[e4 * 4 + 1] = fmaf(xv, wv.y, acc[e4 * 4 + 1]);
                    acc[e4 * 4 + 2] = fmaf(xv, wv.z, acc[e4 * 4 + 2]);
                    acc[e4 * 4 + 3] = fmaf(xv, wv.w, acc[e4 * 4 + 3]);
                }
            }
        }
    } else {
        for (int k = tid; k < d; k += 256) {
            const float xv = to_f32(xr[k]);
            const float* w = Wr + (size_t)k * E;
#pragma unroll
            for (int e = 0; e < EP; ++e)
                if (e < E) acc[e] = fmaf(xv, __ldg(w + e), acc[e]);
        }
    }
#pragma unroll
    for (int e = 0; e < EP; ++e) {
        const float v = warp_sum(acc[e]);
        if (lane == 0) red[warp][e] = v;
    }
    __syncthreads();
    if (warp == 0) {
        float l_lo = 0.f, l_hi = 0.f;
        if (lane < E) {
            l_lo = br ? br[lane] : 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) l_lo += red[w][lane % EP];
        }
        if (EP > 32 && lane + 32 < E) {
            l_hi = br ? br[lane + 32] : 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) l_hi += red[w][(lane + 32) % EP];
        }
        softmax_select_store(l_lo, l_hi, t, q, lane, scores, mask, k_t);
    }
}

// Large T (prefill): a block owns 32 tokens and walks d in chunks staged through shared memory, so
// each router weight is read from L2 once per 32 tokens.  Warp w keeps tokens 4w..4w+3.
template <typename XT, int EP>
__global__ void __launch_bounds__(256) router_tile_kernel(const XT* __restrict__ x, const float* __restrict__ Wr,
                                                          const float* __restrict__ br, float* __restrict__ scores,
                                                          uint64_t* __restrict__ mask, int32_t* __restrict__ k_t,
                                                          int T, int d, SelParams q) {
    constexpr int TB = 32, KC = 64, NE = EP / 32;
    __shared__ __align__(16) float Xs[TB][KC + 4];
    __shared__ float Ws[KC][EP];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t0 = blockIdx.x * TB, E = q.E;
    float acc[4][NE];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int u = 0; u < NE; ++u) acc[i][u] = 0.f;

    for (int k0 = 0; k0 < d; k0 += KC) {
        for (int idx = tid; idx < TB * KC; idx += 256) {
            const int r = idx / KC, c = idx % KC;
            const int t = t0 + r, k = k0 + c;
            Xs[r][c] = (t < T && k < d) ? to_f32(x[(size_t)t * d + k]) : 0.f;
        }
        for (int idx = tid; idx < KC * EP; idx += 256) {
            const int kk = idx / EP, e = idx % EP;
            const int k = k0 + kk;
            Ws[kk][e] = (e < E && k < d) ? __ldg(Wr + (size_t)k * E + e) : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int kk = 0; kk < KC; kk += 4) {
            float4 xv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const float4*>(&Xs[4 * warp + i][kk]);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float w[NE];
#pragma unroll
                for (int v = 0; v < NE; ++v) w[v] = Ws[kk + u][lane + 32 * v];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float xs = u == 0 ? xv[i].x : u == 1 ? xv[i].y : u == 2 ? xv[i].z : xv[i].w;
#pragma unroll
                    for (int v = 0; v < NE; ++v) acc[i][v] = fmaf(xs, w[v], acc[i][v]);
                }
            }
        }
        __syncthreads();
    }
    const float b_lo = (br && lane < E) ? br[lane] : 0.f;
    const float b_hi = (br && NE > 1 && lane + 32 < E) ? br[lane + 32] : 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = t0 + 4 * warp + i;
        if (t < T) {   // uniform across the warp
            const float l_hi = NE > 1 ? acc[i][NE - 1] + b_hi : 0.f;
            softmax_select_store(acc[i][0] + b_lo, l_hi, t, q, lane, scores, mask, k_t);
        }
    }
}

// Selection alone on caller-supplied scores: one warp per token.
__global__ void __launch_bounds__(256) select_kernel(const float* __restrict__ scores, uint64_t* __restrict__ mask,
                                                     int32_t* __restrict__ k_t, int T, SelParams q) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const float s_lo = lane < q.E ? scores[(size_t)t * q.E + lane] : 0.f;
    const float s_hi = lane + 32 < q.E ? scores[(size_t)t * q.E + lane + 32] : 0.f;
    const uint64_t m = select_warp(s_lo, s_hi, q, lane);
    if (lane == 0) {
        mask[t] = m;
        k_t[t] = __popcll(m);
    }
}

// counts[e], offsets[e] and, per chunk of 32 tokens, the number of earlier tokens that selected e
// (chunk_prefix[c,e]).  One block; deterministic; no atomics, so grouped rows come out in token order.
__global__ void __launch_bounds__(1024) finalize_kernel(const uint64_t* __restrict__ mask, int32_t* __restrict__ counts,
                                                        int32_t* __restrict__ offsets, int32_t* __restrict__ chunk_prefix,
                                                        int32_t* __restrict__ counts_out, int T, int E) {
    __shared__ int32_t cnt_s[kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nchunks = (T + kChunk - 1) / kChunk;
    for (int c = warp; c < nchunks; c += 32) {
        const int t = c * kChunk + lane;
        const uint64_t m = t < T ? mask[t] : 0;
        int c_lo = 0, c_hi = 0;
        for (int e = 0; e < E; ++e) {
            const int n = __popc(__ballot_sync(0xffffffffu, (m >> e) & 1));
            if (lane == (e & 31)) {
                if (e < 32) c_lo = n; else c_hi = n;
            }
        }
        if (lane < E) chunk_prefix[(size_t)c * E + lane] = c_lo;
        if (lane + 32 < E) chunk_prefix[(size_t)c * E + lane + 32] = c_hi;
    }
    __syncthreads();
    const int per = (nchunks + 31) / 32;
    for (int e = warp; e < E; e += 32) {
        const int c0 = min(nchunks, lane * per), c1 = min(nchunks, c0 + per);
        int sum = 0;
        for (int c = c0; c < c1; ++c) sum += chunk_prefix[(size_t)c * E + e];
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        int run = incl - sum;
        for (int c = c0; c < c1; ++c) {
            const int v = chunk_prefix[(size_t)c * E + e];
            chunk_prefix[(size_t)c * E + e] = run;
            run += v;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (lane == 0) cnt_s[e] = total;
    }
    __syncthreads();
    if (warp == 0) {
        const int c_lo = lane < E ? cnt_s[lane] : 0;
        const int c_hi = lane + 32 < E ? cnt_s[lane + 32] : 0;
        int i_lo = c_lo, i_hi = c_hi;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int a = __shfl_up_sync(0xffffffffu, i_lo, o);
            const int b = __shfl_up_sync(0xffffffffu, i_hi, o);
            if (lane >= o) {
                i_lo += a;
                i_hi += b;
            }
        }
        const int tot_lo = __shfl_sync(0xffffffffu, i_lo, 31);
        const int tot = tot_lo + __shfl_sync(0xffffffffu, i_hi, 31);
        if (lane < E) {
            counts[lane] = c_lo;
            offsets[lane] = i_lo - c_lo;
            if (counts_out) counts_out[lane] = c_lo;
        }
        if (lane + 32 < E) {
            counts[lane + 32] = c_hi;
            offsets[lane + 32] = tot_lo + i_hi - c_hi;
            if (counts_out) counts_out[lane + 32] = c_hi;
        }
        if (lane == 0) offsets[E] = tot;
    }
}

template <typename XT>
static dsmoe_status launch_router_t(const dsmoe_layer_desc& p, const XT* x, const float* Wr, const float* br,
                                    float* scores, uint64_t* mask, int32_t* k_t, cudaStream_t s) {
    const SelParams q = sel_params(p);
    if (p.T <= 256) {
        if (p.E <= 8) router_small_kernel<XT, 8><<<p.T, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.d, q);
        else if (p.E <= 16) router_small_kernel<XT, 16><<<p.T, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.d, q);
        else if (p.E <= 32) router_small_kernel<XT, 32><<<p.T, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.d, q);
        else router_small_kernel<XT, 64><<<p.T, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.d, q);
    } else {
        const int grid = ceil_div(p.T, 32);
        if (p.E <= 32) router_tile_kernel<XT, 32><<<grid, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q);
        else router_tile_kernel<XT, 64><<<grid, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q);
    }
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_router(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                           float* scores, uint64_t* mask, int32_t* k_t, cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    if (p.dtype == DSMOE_BF16)
        return launch_router_t(p, static_cast<const __nv_bfloat16*>(x), Wr, br, scores, mask, k_t, s);
    return launch_router_t(p, static_cast<const float*>(x), Wr, br, scores, mask, k_t, s);
}

dsmoe_status launch_select(const dsmoe_layer_desc& p, const float* scores, uint64_t* mask, int32_t* k_t,
                           cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    select_kernel<<<ceil_div(p.T, 8), 256, 0, s>>>(scores, mask, k_t, p.T, sel_params(p));
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_finalize(const dsmoe_layer_desc& p, const uint64_t* mask, int32_t* counts, int32_t* offsets,
                             int32_t* chunk_prefix, int32_t* counts_out, cudaStream_t s) {
    finalize_kernel<<<1, 1024, 0, s>>>(mask, counts, offsets, chunk_prefix, counts_out, p.T, p.E);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace dsmoe
