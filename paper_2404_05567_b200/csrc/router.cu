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
    return SelParams{p.E, p.mode, p.eps, p.eps_normalized, p.K, p.min_k, nullptr};
}

// Small T (decode): a block per TT tokens (1, or 4 (2 beyond 32 experts) from 64 tokens on: the tokens of a block share its loads of Wr, which
// every block reads in full out of L2), the reduction over d split across all 256 threads.  A token's sums are formed
// in the same order whatever TT is.
template <typename XT, int EP, int TT>
__global__ void __launch_bounds__(256) router_small_kernel(const XT* __restrict__ x, const float* __restrict__ Wr,
                                                           const float* __restrict__ br, float* __restrict__ scores,
                                                           uint64_t* __restrict__ mask, int32_t* __restrict__ k_t,
                                                           int T, int d, SelParams q) {
    __shared__ float red[TT][8][EP];
    const int t0 = blockIdx.x * TT, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int E = q.E;
    float acc[TT][EP];
#pragma unroll
    for (int u = 0; u < TT; ++u)
#pragma unroll
        for (int e = 0; e < EP; ++e) acc[u][e] = 0.f;
    const XT* xr[TT];
#pragma unroll
    for (int u = 0; u < TT; ++u) xr[u] = x + (size_t)min(t0 + u, T - 1) * d;     // past the end: the last token again, unused
    if ((E & 3) == 0) {
        for (int k = tid; k < d; k += 256) {
            float xv[TT];
#pragma unroll
            for (int u = 0; u < TT; ++u) xv[u] = to_f32(xr[u][k]);
            const float4* w = reinterpret_cast<const float4*>(Wr + (size_t)k * E);
#pragma unroll
            for (int e4 = 0; e4 < EP / 4; ++e4) {
                if (e4 * 4 < E) {
                    const float4 wv = __ldg(w + e4);
#pragma unroll
                    for (int u = 0; u < TT; ++u) {
                        acc[u][e4 * 4 + 0] = fmaf(xv[u], wv.x, acc[u][e4 * 4 + 0]);
                        acc[u][e4 * 4 + 1] = fmaf(xv[u], wv.y, acc[u][e4 * 4 + 1]);
                        acc[u][e4 * 4 + 2] = fmaf(xv[u], wv.z, acc[u][e4 * 4 + 2]);
                        acc[u][e4 * 4 + 3] = fmaf(xv[u], wv.w, acc[u][e4 * 4 + 3]);
                    }
                }
            }
        }
    } else {
        for (int k = tid; k < d; k += 256) {
            float xv[TT];
#pragma unroll
            for (int u = 0; u < TT; ++u) xv[u] = to_f32(xr[u][k]);
            const float* w = Wr + (size_t)k * E;
#pragma unroll
            for (int e = 0; e < EP; ++e) {
                if (e < E) {
                    const float wv = __ldg(w + e);
#pragma unroll
                    for (int u = 0; u < TT; ++u) acc[u][e] = fmaf(xv[u], wv, acc[u][e]);
                }
            }
        }
    }
#pragma unroll
    for (int u = 0; u < TT; ++u) {
#pragma unroll
        for (int e = 0; e < EP; ++e) {
            const float v = warp_sum(acc[u][e]);
            if (lane == 0) red[u][warp][e] = v;
        }
    }
    __syncthreads();
    if (warp < TT && t0 + warp < T) {
        const int u = warp;
        float l_lo = 0.f, l_hi = 0.f;
        if (lane < E) {
            l_lo = br ? br[lane] : 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) l_lo += red[u][w][lane % EP];
        }
        if (EP > 32 && lane + 32 < E) {
            l_hi = br ? br[lane + 32] : 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) l_hi += red[u][w][(lane + 32) % EP];
        }
        softmax_select_store(l_lo, l_hi, t0 + u, q, lane, scores, mask, k_t);
    }
}

// Large T (prefill): an fp32 FMA GEMM [T,d] x [d,E] with the softmax and the selection as its epilogue.  A block
// owns 64 tokens and walks d in chunks of 128 staged through shared memory (two buffers; the next chunk's global
// loads are in flight while the current one is multiplied).  A thread keeps 2 tokens x EPL experts (EPL = 4 for
// E <= 32, 8 for E <= 64): 8 neighbouring lanes cover all experts of a token with 16-byte shared-memory reads that
// the lanes of a warp share, so the loop is bound by the FMA pipe, not by shared-memory traffic.
//   warp w (of a group of 8): tokens 8w..8w+7; lane: tokens 8w + lane/8 + {0, 4}; experts 4 (lane % 8) + {0..3}
//   (and 32 + the same when EPL = 8)
template <typename XT>
__device__ __forceinline__ void load8_as_f32(const XT* p, bool vec, int nvalid, float (&out)[8]);
template <>
__device__ __forceinline__ void load8_as_f32<__nv_bfloat16>(const __nv_bfloat16* p, bool vec, int nvalid, float (&out)[8]) {
    if (vec && nvalid == 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            out[2 * i] = f.x;
            out[2 * i + 1] = f.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = i < nvalid ? __bfloat162float(p[i]) : 0.f;
    }
}
template <>
__device__ __forceinline__ void load8_as_f32<float>(const float* p, bool vec, int nvalid, float (&out)[8]) {
    if (vec && nvalid == 8) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = i < nvalid ? p[i] : 0.f;
    }
}

constexpr int kRtTB = 64, kRtKC = 128, kRtXS = kRtKC + 4, kRtSplit = 4, kRtThreads = 256 * kRtSplit;
template <int EPL>
constexpr size_t router_tile_smem() {
    return (size_t)2 * kRtTB * kRtXS * sizeof(float) + (size_t)2 * kRtKC * (8 * EPL) * sizeof(float);
}

// 1024 threads: four groups of 8 warps; group g multiplies the g-th quarter of every 128-wide chunk (the same 2 x EPL
// tile per thread in each group), so that every scheduler has 8 warps to hide the FMA and shared-memory latencies
// behind.  The groups' partial sums meet in shared memory at the end and are added in group order.
template <typename XT, int EPL>
__global__ void __launch_bounds__(kRtThreads, 1) router_tile_kernel(const XT* __restrict__ x, const float* __restrict__ Wr,
                                                                    const float* __restrict__ br, float* __restrict__ scores,
                                                                    uint64_t* __restrict__ mask, int32_t* __restrict__ k_t,
                                                                    int T, int d, SelParams q) {
    constexpr int TB = kRtTB, KC = kRtKC, EP = 8 * EPL, XS = kRtXS, NT = kRtThreads;
    constexpr int NW = KC * EP / NT, NX = TB * KC / 8 / NT, KQ = KC / kRtSplit;
    static_assert(NX == 1 && NW >= 1, "staging: one 8-element group of x per thread");
    extern __shared__ __align__(16) float rt_smem[];
    float (*Xs)[TB][XS] = reinterpret_cast<float (*)[TB][XS]>(rt_smem);                      // [2][TB][XS]
    float (*Ws)[KC][EP] = reinterpret_cast<float (*)[KC][EP]>(rt_smem + 2 * TB * XS);          // [2][KC][EP]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t0 = blockIdx.x * TB, E = q.E;
    const bool vec = (d & 7) == 0;                    // rows of x start 16-byte aligned
    // staging: thread -> 8 consecutive k of one token (16 threads per token row), and NW router weights
    const int xr = tid >> 4, xc = (tid & 15) * 8;
    const XT* xrow = x + (size_t)min(t0 + xr, T - 1) * d;
    const bool xrow_ok = t0 + xr < T;
    float xreg[8], wreg[NW];
    auto fetch = [&](int k0) {
        const int nv = xrow_ok ? max(0, min(8, d - (k0 + xc))) : 0;
        if (nv > 0) load8_as_f32<XT>(xrow + k0 + xc, vec, nv, xreg);
        else {
#pragma unroll
            for (int i = 0; i < 8; ++i) xreg[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            const int idx = tid + i * NT, kk = idx / EP, e = idx % EP;
            wreg[i] = (e < E && k0 + kk < d) ? __ldg(Wr + (size_t)(k0 + kk) * E + e) : 0.f;
        }
    };
    auto stash = [&](int b) {
        *reinterpret_cast<float4*>(&Xs[b][xr][xc]) = make_float4(xreg[0], xreg[1], xreg[2], xreg[3]);
        *reinterpret_cast<float4*>(&Xs[b][xr][xc + 4]) = make_float4(xreg[4], xreg[5], xreg[6], xreg[7]);
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            const int idx = tid + i * NT;
            Ws[b][idx / EP][idx % EP] = wreg[i];
        }
    };
    const int grp = warp >> 3, w8 = warp & 7;
    const int tk = w8 * 8 + (lane >> 3), eo = (lane & 7) * 4;   // this thread's first token (in the block), first expert
    float acc[2][EPL];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int u = 0; u < EPL; ++u) acc[i][u] = 0.f;

    fetch(0);
    stash(0);
    __syncthreads();
    int b = 0;
    for (int k0 = 0; k0 < d; k0 += KC) {
        const bool more = k0 + KC < d;
        if (more) fetch(k0 + KC);
#pragma unroll
        for (int kq = 0; kq < KQ; kq += 4) {
            const int kk = grp * KQ + kq;
            const float4 xa = *reinterpret_cast<const float4*>(&Xs[b][tk][kk]);
            const float4 xb = *reinterpret_cast<const float4*>(&Xs[b][tk + 4][kk]);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float xs0 = u == 0 ? xa.x : u == 1 ? xa.y : u == 2 ? xa.z : xa.w;
                const float xs1 = u == 0 ? xb.x : u == 1 ? xb.y : u == 2 ? xb.z : xb.w;
#pragma unroll
                for (int h = 0; h < EPL / 4; ++h) {
                    const float4 w = *reinterpret_cast<const float4*>(&Ws[b][kk + u][eo + 32 * h]);
                    acc[0][4 * h + 0] = fmaf(xs0, w.x, acc[0][4 * h + 0]);
                    acc[0][4 * h + 1] = fmaf(xs0, w.y, acc[0][4 * h + 1]);
                    acc[0][4 * h + 2] = fmaf(xs0, w.z, acc[0][4 * h + 2]);
                    acc[0][4 * h + 3] = fmaf(xs0, w.w, acc[0][4 * h + 3]);
                    acc[1][4 * h + 0] = fmaf(xs1, w.x, acc[1][4 * h + 0]);
                    acc[1][4 * h + 1] = fmaf(xs1, w.y, acc[1][4 * h + 1]);
                    acc[1][4 * h + 2] = fmaf(xs1, w.z, acc[1][4 * h + 2]);
                    acc[1][4 * h + 3] = fmaf(xs1, w.w, acc[1][4 * h + 3]);
                }
            }
        }
        if (more) stash(b ^ 1);
        __syncthreads();
        b ^= 1;
    }
    // the groups' partial logits -> shared memory as [group][token][expert] (all staging buffers are free now), then
    // one warp per token adds them in group order
    float* Ls = rt_smem;                            // kRtSplit x TB x EP floats
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int h = 0; h < EPL / 4; ++h)
            *reinterpret_cast<float4*>(&Ls[(grp * TB + tk + 4 * i) * EP + eo + 32 * h]) =
                make_float4(acc[i][4 * h], acc[i][4 * h + 1], acc[i][4 * h + 2], acc[i][4 * h + 3]);
    __syncthreads();
    const float b_lo = (br && lane < E) ? br[lane] : 0.f;
    const float b_hi = (br && lane + 32 < E) ? br[lane + 32] : 0.f;
    for (int tl = warp; tl < TB; tl += NT / 32) {
        const int t = t0 + tl;
        if (t < T) {   // uniform across the warp
            float l_lo = b_lo, l_hi = b_hi;
#pragma unroll
            for (int g = 0; g < kRtSplit; ++g) {
                l_lo += Ls[(g * TB + tl) * EP + lane];
                if (EP > 32) l_hi += Ls[(g * TB + tl) * EP + (lane + 32) % EP];
            }
            softmax_select_store(l_lo, l_hi, t, q, lane, scores, mask, k_t);
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
// (chunk_prefix[c,e]).  Deterministic; no atomics, so grouped rows come out in token order.  Two kernels:
// chunk_count_kernel, one warp per chunk (lane = token, one ballot per expert), leaves the chunk's counts in
// chunk_prefix[c,:]; finalize_kernel, one block, turns them into exclusive prefixes over the chunks (warp e scans
// expert e, 32 chunks per warp-wide scan) and writes the totals and their offsets.
__global__ void __launch_bounds__(256) chunk_count_kernel(const uint64_t* __restrict__ mask, int32_t* __restrict__ chunk_prefix,
                                                          int T, int E) {
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (c * kChunk >= T) return;
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

__global__ void __launch_bounds__(1024) finalize_kernel(int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                                        int32_t* __restrict__ chunk_prefix, int32_t* __restrict__ counts_out,
                                                        int T, int E) {
    __shared__ int32_t cnt_s[kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nchunks = (T + kChunk - 1) / kChunk;
    for (int e = warp; e < E; e += 32) {
        int carry = 0;
        for (int c0 = 0; c0 < nchunks; c0 += 32 * 4) {
            // four scans' worth of loads are issued together
            int v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = c0 + 32 * j + lane;
                v[j] = c < nchunks ? chunk_prefix[(size_t)c * E + e] : 0;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = c0 + 32 * j + lane;
                int incl = v[j];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int u = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += u;
                }
                if (c < nchunks) chunk_prefix[(size_t)c * E + e] = carry + incl - v[j];
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        if (lane == 0) cnt_s[e] = carry;
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
#define ROUTER_SMALL(EP, TT)                                                                                            \
    do {                                                                                                                \
        if (p.T >= 64)                                                                                                  \
            router_small_kernel<XT, EP, TT><<<ceil_div(p.T, TT), 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q); \
        else                                                                                                            \
            router_small_kernel<XT, EP, 1><<<p.T, 256, 0, s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q);             \
    } while (0)
        if (p.E <= 8) ROUTER_SMALL(8, 4);
        else if (p.E <= 16) ROUTER_SMALL(16, 4);
        else if (p.E <= 32) ROUTER_SMALL(32, 4);
        else ROUTER_SMALL(64, 2);                 // 2 x 64 sums a thread: four tokens' would not fit the registers
#undef ROUTER_SMALL
    } else {
        const int grid = ceil_div(p.T, kRtTB);
        DeviceState* st = nullptr;
        DSMOE_TRY(device_state(&st));
        bool& attr_set = sizeof(XT) == 4 ? st->attr_router_f32 : st->attr_router_bf16;
        if (!attr_set) {
            DSMOE_CUDA_TRY(cudaFuncSetAttribute(router_tile_kernel<XT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)router_tile_smem<4>()));
            DSMOE_CUDA_TRY(cudaFuncSetAttribute(router_tile_kernel<XT, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)router_tile_smem<8>()));
            attr_set = true;
        }
        if (p.E <= 32)
            router_tile_kernel<XT, 4><<<grid, kRtThreads, router_tile_smem<4>(), s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q);
        else
            router_tile_kernel<XT, 8><<<grid, kRtThreads, router_tile_smem<8>(), s>>>(x, Wr, br, scores, mask, k_t, p.T, p.d, q);
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

// Threshold-TopK ("Expert Sampling Strategy" paragraph): K = the batch average of the per-token counts that the
// threshold gave, rounded half up and kept within [1, E].  One block; integer sums, so the result does not depend
// on the order of the additions.
__global__ void __launch_bounds__(1024) batch_k_kernel(const int32_t* __restrict__ k_t, int T, int E, int* __restrict__ K_out) {
    __shared__ long long part[32];
    long long sum = 0;
    for (int t = threadIdx.x; t < T; t += 1024) sum += k_t[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long total = 0;
        for (int w = 0; w < 32; ++w) total += part[w];
        long long k = (2 * total + T) / (2ll * T);
        *K_out = (int)(k < 1 ? 1 : (k > E ? E : k));
    }
}

dsmoe_status launch_select(const dsmoe_layer_desc& p, const float* scores, uint64_t* mask, int32_t* k_t,
                           cudaStream_t s, int* k_scratch) {
    if (p.T == 0) return DSMOE_OK;
    SelParams q = sel_params(p);
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) {
        if (!k_scratch) return DSMOE_ERR_UNSUPPORTED;
        q.mode = DSMOE_SELECT_THRESHOLD;
        q.min_k = 0;                     // the counts are the threshold's own
        select_kernel<<<ceil_div(p.T, 8), 256, 0, s>>>(scores, mask, k_t, p.T, q);
        DSMOE_CUDA_TRY(cudaGetLastError());
        batch_k_kernel<<<1, 1024, 0, s>>>(k_t, p.T, p.E, k_scratch);
        DSMOE_CUDA_TRY(cudaGetLastError());
        q.mode = DSMOE_SELECT_TOPK;
        q.min_k = p.min_k;
        q.K_dev = k_scratch;
    }
    select_kernel<<<ceil_div(p.T, 8), 256, 0, s>>>(scores, mask, k_t, p.T, q);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_chunk_counts(const dsmoe_layer_desc& p, const uint64_t* mask, int32_t* chunk_prefix, cudaStream_t s) {
    const int nchunks = ceil_div(p.T, kChunk);
    if (nchunks > 0) {
        chunk_count_kernel<<<ceil_div(nchunks, 8), 256, 0, s>>>(mask, chunk_prefix, p.T, p.E);
        DSMOE_CUDA_TRY(cudaGetLastError());
    }
    return DSMOE_OK;
}

dsmoe_status launch_chunk_scan(const dsmoe_layer_desc& p, int32_t* counts, int32_t* offsets, int32_t* chunk_prefix,
                               int32_t* counts_out, cudaStream_t s) {
    finalize_kernel<<<1, 1024, 0, s>>>(counts, offsets, chunk_prefix, counts_out, p.T, p.E);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_finalize(const dsmoe_layer_desc& p, const uint64_t* mask, int32_t* counts, int32_t* offsets,
                             int32_t* chunk_prefix, int32_t* counts_out, cudaStream_t s) {
    DSMOE_TRY(launch_chunk_counts(p, mask, chunk_prefix, s));
    return launch_chunk_scan(p, counts, offsets, chunk_prefix, counts_out, s);
}

}  // namespace dsmoe
