// Grouping of tokens by expert and the router-weighted aggregation back into token order -- the
// "duplication of intermediate tokens and the aggregation of outputs" that the paper's GPU
// Inference Analysis names as the overhead of sparse inference -- plus the one-off weight packer.
#include <algorithm>

#include "common.cuh"

namespace dsmoe {

// Row indices.  A warp owns a chunk of 32 consecutive tokens; for expert e the ballot of "selected"
// gives each token its rank inside the chunk, and chunk_prefix gives the number of earlier tokens,
// so rows inside an expert segment ascend by token without any atomic.
// SCAN 1: chunk_prefix holds the chunks' own counts (chunk_count_kernel's output, not yet the prefixes over the
// chunks): every block adds up the chunks before its own and all chunks itself -- a few thousand integers out of
// L2 -- instead of waiting for a one-block scan kernel in between; block 0 writes counts, offsets (and counts_out).
// SCAN 2 (at most kCountInBlockChunks chunks): every block also counts the chunks itself, from the masks.
// The integers are the same either way.
constexpr int kCountInBlockChunks = 8;
template <int SCAN>
__global__ void __launch_bounds__(128) permute_index_kernel(const uint64_t* __restrict__ mask,
                                                            const float* __restrict__ scores,
                                                            int32_t* __restrict__ offsets,
                                                            const int32_t* __restrict__ chunk_prefix,
                                                            int32_t* __restrict__ counts, int32_t* __restrict__ counts_out,
                                                            int32_t* __restrict__ row_token, float* __restrict__ row_gate,
                                                            int32_t* __restrict__ token_rows, int T, int E, int W,
                                                            int64_t amax, uint4* __restrict__ zero_out, int row_vecs) {
    // a chunk's scores, staged so that the loop over the experts below waits for no load: [token][E + 1]
    __shared__ float sc_s[4][kChunk * (kMaxExperts + 1)];
    __shared__ int before_s[4][kMaxExperts], total_s[4][kMaxExperts], base_s[4][kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c0 = blockIdx.x * 4, c = c0 + warp;
    const int nchunks = (T + kChunk - 1) / kChunk;
    const bool live = c < nchunks;
    const int t = c * kChunk + lane;
    const uint64_t m = live && t < T ? mask[t] : 0;
    if (live) {
        float* sc = sc_s[warp];
        const float* src = scores + (size_t)c * kChunk * E;
        const int n = min(kChunk, T - c * kChunk) * E;
        int row = lane / E, col = lane % E;             // of element i below, kept up without a division per element
#pragma unroll 1
        for (int i0 = lane; i0 < n; i0 += 32 * 8) {      // eight coalesced loads under way at a time
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = i0 + 32 * j < n ? __ldg(src + i0 + 32 * j) : 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (i0 + 32 * j < n) sc[row * (E + 1) + col] = v[j];
                col += 32;
                while (col >= E) {
                    col -= E;
                    ++row;
                }
            }
        }
    }
    __shared__ int cnt_s[SCAN == 2 ? kCountInBlockChunks : 1][kMaxExperts];
    if (SCAN == 2) {
        for (int k = warp; k < nchunks; k += 4) {
            const int tk = k * kChunk + lane;
            const uint64_t mk = tk < T ? mask[tk] : 0;
            int n_lo = 0, n_hi = 0;
            for (int e = 0; e < E; ++e) {
                const int n = __popc(__ballot_sync(0xffffffffu, (mk >> e) & 1));
                if (lane == (e & 31)) {
                    if (e < 32) n_lo = n; else n_hi = n;
                }
            }
            cnt_s[k][lane] = n_lo;
            cnt_s[k][lane + 32] = n_hi;
        }
        __syncthreads();
    }
    const auto chunk_count = [&](int k, int e) { return SCAN == 2 ? cnt_s[k][e] : chunk_prefix[(size_t)k * E + e]; };
    if (SCAN) {
        // thread (e, part) adds every `parts`-th chunk's count of expert e: coalesced rows of E integers
        const int EP = E <= 32 ? 32 : 64, parts = 128 / EP;
        const int e = threadIdx.x % EP, part = threadIdx.x / EP;
        int before = 0, total = 0;
        if (e < E) {
            // sixteen loads are issued before the first one is used
#pragma unroll 1
            for (int k0 = part; k0 < nchunks; k0 += parts * 16) {
                int v[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int k = k0 + j * parts;
                    v[j] = k < nchunks ? chunk_count(k, e) : 0;
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    total += v[j];
                    if (k0 + j * parts < c0) before += v[j];
                }
            }
        }
        before_s[part][e] = before;
        total_s[part][e] = total;
        // the block's own chunks' counts (warp 0 needs them below): asked for before the barrier
        int own_lo[4] = {0, 0, 0, 0}, own_hi[4] = {0, 0, 0, 0};
        if (warp == 0) {
#pragma unroll
            for (int w = 0; w < 3; ++w) {
                if (c0 + w < nchunks) {
                    if (lane < E) own_lo[w] = chunk_count(c0 + w, lane);
                    if (lane + 32 < E) own_hi[w] = chunk_count(c0 + w, lane + 32);
                }
            }
        }
        __syncthreads();
        if (warp == 0) {
            int b_lo = 0, b_hi = 0, c_lo = 0, c_hi = 0;
            for (int k = 0; k < parts; ++k) {
                b_lo += before_s[k][lane];
                c_lo += total_s[k][lane];
                if (EP == 64) {
                    b_hi += before_s[k][lane + 32];
                    c_hi += total_s[k][lane + 32];
                }
            }
            if (lane >= E) c_lo = 0;
            if (lane + 32 >= E) c_hi = 0;
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
            int run_lo = i_lo - c_lo + b_lo, run_hi = tot_lo + i_hi - c_hi + b_hi;   // first row of chunk c0 in the expert
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                base_s[w][lane] = run_lo;
                base_s[w][lane + 32] = run_hi;
                run_lo += own_lo[w];
                run_hi += own_hi[w];
            }
            if (blockIdx.x == 0) {
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
        __syncthreads();
    }
    if (!live) return;
    __syncwarp();
    // lane l holds the first row of this chunk in experts l and l + 32 (passed around by shuffles)
    int base_lo, base_hi;
    if (SCAN) {
        base_lo = base_s[warp][lane];
        base_hi = base_s[warp][lane + 32];
    } else {
        base_lo = lane < E ? offsets[lane] + chunk_prefix[(size_t)c * E + lane] : 0;
        base_hi = lane + 32 < E ? offsets[lane + 32] + chunk_prefix[(size_t)c * E + lane + 32] : 0;
    }
    // From here a lane stands for experts `lane` and `lane + 32` and the warp walks the chunk's tokens in order: an
    // expert's rows ascend by token, a lane counts its own rows, and nothing is exchanged between lanes but the
    // token's selection word.  (A lane per token and a ballot per expert cost three times the instructions.)
    const float* sc = sc_s[warp];
    const uint32_t m_lo = (uint32_t)m, m_hi = (uint32_t)(m >> 32);
    const uint32_t below = (1u << lane) - 1u;
    const bool e_lo = lane < E, e_hi = lane + 32 < E;
    const int ntok = min(kChunk, T - c * kChunk);
    int row_lo = base_lo, row_hi = base_hi;
    for (int tt = 0; tt < ntok; ++tt) {
        const uint32_t a = __shfl_sync(0xffffffffu, m_lo, tt);
        const int tok = c * kChunk + tt;
        if (e_lo && ((a >> lane) & 1u)) {
            const int r = row_lo++;
            const int slot = __popc(a & below);
            if (r >= 0 && r < amax) {   // inconsistent caller-supplied offsets must not become a wild store
                row_token[r] = tok;
                row_gate[r] = sc[tt * (E + 1) + lane];
            }
            if (slot < W) token_rows[(size_t)tok * W + slot] = r;
        }
        if (E > 32) {
            const uint32_t b = __shfl_sync(0xffffffffu, m_hi, tt);
            if (e_hi && ((b >> lane) & 1u)) {
                const int r = row_hi++;
                const int slot = __popc(a) + __popc(b & below);
                if (r >= 0 && r < amax) {
                    row_token[r] = tok;
                    row_gate[r] = sc[tt * (E + 1) + lane + 32];
                }
                if (slot < W) token_rows[(size_t)tok * W + slot] = r;
            }
        }
    }
    if (t < T)
        for (int slot = __popcll(m); slot < W; ++slot) token_rows[(size_t)t * W + slot] = -1;
    if (zero_out) {
        // Eq. 1 with an empty selection is the zero vector: no expert tile will ever write this token's row
        unsigned none = __ballot_sync(0xffffffffu, t < T && m == 0);
        while (none) {
            const int l = __ffs(none) - 1;
            none &= none - 1;
            uint4* row = zero_out + (size_t)(c * kChunk + l) * row_vecs;
            for (int v = lane; v < row_vecs; v += 32) row[v] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

// xp[r,:] = x[row_token[r],:] for r < A, 16 bytes per lane per step, one warp per row.
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ row_token,
                                                          const int32_t* __restrict__ offsets, uint4* __restrict__ xp,
                                                          int E, int T, int vec_per_row, int64_t amax) {
    const int64_t A = min((int64_t)offsets[E], amax);
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * 8;
    for (int64_t r = blockIdx.x * 8 + (threadIdx.x >> 5); r < A; r += warps) {
        const int t = row_token[r];
        if ((unsigned)t >= (unsigned)T) continue;   // never trust an index blindly
        const uint4* src = x + (size_t)t * vec_per_row;
        uint4* dst = xp + (size_t)r * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32) dst[v] = __ldg(src + v);
    }
}

__device__ __forceinline__ void fma8(float (&acc)[8], const uint4 v, float g) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        acc[2 * i] = fmaf(g, f.x, acc[2 * i]);
        acc[2 * i + 1] = fmaf(g, f.y, acc[2 * i + 1]);
    }
}

// out[t,:] = sum_i gate[r_i] * yp[r_i,:] in ascending expert order, fp32, one rounding.  Block per token.
template <bool OUT_F32>
__global__ void __launch_bounds__(128) combine_bf16_kernel(const uint4* __restrict__ yp, const float* __restrict__ row_gate,
                                                           const int32_t* __restrict__ token_rows,
                                                           const int32_t* __restrict__ k_t, void* __restrict__ out,
                                                           int d, int W, int64_t amax) {
    __shared__ int32_t rows_s[kMaxExperts];
    __shared__ float gate_s[kMaxExperts];
    const int t = blockIdx.x;
    const int k = max(0, min(k_t[t], W));
    if ((int)threadIdx.x < k) {
        const int r = token_rows[(size_t)t * W + threadIdx.x];
        const bool ok = r >= 0 && r < amax;
        rows_s[threadIdx.x] = ok ? r : 0;
        gate_s[threadIdx.x] = ok ? row_gate[r] : 0.f;
    }
    __syncthreads();
    const int nvec = d / 8;
    for (int v = blockIdx.y * 128 + threadIdx.x; v < nvec; v += 128 * gridDim.y) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        // four rows' loads are issued before their first use (past the k-th row, row 0 is fetched again and not used)
        for (int i = 0; i < k; i += 4) {
            uint4 y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) y[j] = __ldg(yp + (size_t)rows_s[i + j < k ? i + j : 0] * nvec + v);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (i + j < k) fma8(acc, y[j], gate_s[i + j]);
        }
        if (OUT_F32) {
            float4* o = reinterpret_cast<float4*>(out) + ((size_t)t * nvec + v) * 2;
            o[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            o[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
        } else {
            uint4 pk;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
            for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            reinterpret_cast<uint4*>(out)[(size_t)t * nvec + v] = pk;
        }
    }
}

// fp32 rows: the plain path's fp32 layers (gates applied here) and the tensor-core path's gate-weighted fp32 expert
// outputs (row_gate == NULL: only the sum is left to do; the output may be bf16)
template <bool OUT_BF16>
__global__ void __launch_bounds__(128) combine_f32_kernel(const float4* __restrict__ yp, const float* __restrict__ row_gate,
                                                          const int32_t* __restrict__ token_rows,
                                                          const int32_t* __restrict__ k_t, void* __restrict__ out,
                                                          int d, int W, int64_t amax) {
    __shared__ int32_t rows_s[kMaxExperts];
    __shared__ float gate_s[kMaxExperts];
    const int t = blockIdx.x;
    const int k = max(0, min(k_t[t], W));
    if ((int)threadIdx.x < k) {
        const int r = token_rows[(size_t)t * W + threadIdx.x];
        const bool ok = r >= 0 && r < amax;
        rows_s[threadIdx.x] = ok ? r : 0;
        gate_s[threadIdx.x] = !ok ? 0.f : row_gate ? row_gate[r] : 1.f;
    }
    __syncthreads();
    const int nvec = d / 4;
    for (int v = blockIdx.y * 128 + threadIdx.x; v < nvec; v += 128 * gridDim.y) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        // four rows' loads are issued before their first use (past the k-th row, row 0 is fetched again and not used)
        for (int i = 0; i < k; i += 4) {
            float4 y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) y[j] = __ldg(yp + (size_t)rows_s[i + j < k ? i + j : 0] * nvec + v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (i + j >= k) continue;
                const float g = gate_s[i + j];
                acc.x = fmaf(g, y[j].x, acc.x);
                acc.y = fmaf(g, y[j].y, acc.y);
                acc.z = fmaf(g, y[j].z, acc.z);
                acc.w = fmaf(g, y[j].w, acc.w);
            }
        }
        if (OUT_BF16) {
            uint2 pk;
            *reinterpret_cast<__nv_bfloat162*>(&pk.x) = __floats2bfloat162_rn(acc.x, acc.y);
            *reinterpret_cast<__nv_bfloat162*>(&pk.y) = __floats2bfloat162_rn(acc.z, acc.w);
            reinterpret_cast<uint2*>(out)[(size_t)t * nvec + v] = pk;
        } else {
            reinterpret_cast<float4*>(out)[(size_t)t * nvec + v] = acc;
        }
    }
}

// Packing of a batch of [rows = reduction, cols = outputs] bf16 matrices: dst[b][r / 64][c][r % 64] = src[b][r][c]
// (32x32 tiles through smem; rows is a multiple of 64 where this layout is used).
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ src,
                                                             __nv_bfloat16* __restrict__ dst, int rows, int cols) {
    __shared__ __nv_bfloat16 tile[32][33];
    const size_t base = (size_t)blockIdx.z * rows * cols;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        if (r < rows && c < cols) tile[i][tx] = src[base + (size_t)r * cols + c];
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;
        if (r < rows && c < cols) dst[base + ((size_t)(r / 64) * cols + c) * 64 + (r % 64)] = tile[tx][i];
    }
}

dsmoe_status launch_permute(const dsmoe_layer_desc& p, const void* x, const float* scores, const uint64_t* mask,
                            const int32_t* offsets, const int32_t* chunk_prefix, int32_t* row_token, float* row_gate,
                            int32_t* token_rows, void* xp, cudaStream_t s, void* zero_out) {
    if (p.T == 0) return DSMOE_OK;
    const int nchunks = ceil_div(p.T, kChunk);
    const int64_t amax = (int64_t)amax_of(p);
    const int row_vecs = (int)((size_t)p.d * (p.out_fp32 ? 4 : elem_size(p.dtype)) / 16);
    permute_index_kernel<0><<<ceil_div(nchunks, 4), 128, 0, s>>>(mask, scores, const_cast<int32_t*>(offsets), chunk_prefix,
                                                                    nullptr, nullptr, row_token, row_gate, token_rows, p.T,
                                                                    p.E, width_of(p), amax, static_cast<uint4*>(zero_out),
                                                                    row_vecs);
    DSMOE_CUDA_TRY(cudaGetLastError());
    if (xp) {
        const int vec_per_row = (int)((size_t)p.d * elem_size(p.dtype) / 16);
        const int grid = (int)(amax / 8 + 1 < 148 * 16 ? amax / 8 + 1 : 148 * 16);
        gather_rows_kernel<<<grid, 256, 0, s>>>(static_cast<const uint4*>(x), row_token, offsets,
                                                static_cast<uint4*>(xp), p.E, p.T, vec_per_row, amax);
        DSMOE_CUDA_TRY(cudaGetLastError());
    }
    return DSMOE_OK;
}

// Up to this many chunks every block of permute_index_kernel adds up the chunks' counts itself (no scan kernel)
constexpr int kScanInBlockChunks = 512;

dsmoe_status launch_group(const dsmoe_layer_desc& p, const float* scores, const uint64_t* mask, int32_t* counts,
                          int32_t* offsets, int32_t* chunk_prefix, int32_t* counts_out, int32_t* row_token,
                          float* row_gate, int32_t* token_rows, cudaStream_t s, void* zero_out, bool chunk_counts_ready) {
    const int nchunks = ceil_div(p.T, kChunk);
    const int row_vecs = (int)((size_t)p.d * (p.out_fp32 ? 4 : elem_size(p.dtype)) / 16);
    if (nchunks > 0 && nchunks <= kCountInBlockChunks) {
        permute_index_kernel<2><<<ceil_div(nchunks, 4), 128, 0, s>>>(mask, scores, offsets, nullptr, counts, counts_out,
                                                                    row_token, row_gate, token_rows, p.T, p.E, width_of(p),
                                                                    (int64_t)amax_of(p), static_cast<uint4*>(zero_out),
                                                                    row_vecs);
        DSMOE_CUDA_TRY(cudaGetLastError());
        return DSMOE_OK;
    }
    if (!chunk_counts_ready) DSMOE_TRY(launch_chunk_counts(p, mask, chunk_prefix, s));
    if (nchunks == 0 || nchunks > kScanInBlockChunks) {
        DSMOE_TRY(launch_chunk_scan(p, counts, offsets, chunk_prefix, counts_out, s));
        return launch_permute(p, nullptr, scores, mask, offsets, chunk_prefix, row_token, row_gate, token_rows, nullptr, s,
                              zero_out);
    }
    permute_index_kernel<1><<<ceil_div(nchunks, 4), 128, 0, s>>>(mask, scores, offsets, chunk_prefix, counts, counts_out,
                                                                   row_token, row_gate, token_rows, p.T, p.E, width_of(p),
                                                                   (int64_t)amax_of(p), static_cast<uint4*>(zero_out),
                                                                   row_vecs);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_combine(const dsmoe_layer_desc& p, const void* yp, const float* row_gate, const int32_t* token_rows,
                            const int32_t* k_t, void* out, cudaStream_t s, bool yp_f32) {
    if (p.T == 0) return DSMOE_OK;
    const int W = width_of(p);
    const int64_t amax = (int64_t)amax_of(p);
    // with few tokens a row's columns are shared out over several blocks (blockIdx.y), enough to cover the SMs
    const int col_blocks = ceil_div(p.d / (yp_f32 || p.dtype != DSMOE_BF16 ? 4 : 8), 128);
    const dim3 grid(p.T, (unsigned)(std::max(1, std::min(col_blocks, 1024 / p.T))));
    if (yp_f32 && p.dtype == DSMOE_BF16 && !p.out_fp32) {
        combine_f32_kernel<true><<<grid, 128, 0, s>>>(static_cast<const float4*>(yp), row_gate, token_rows, k_t, out, p.d, W, amax);
    } else if (yp_f32) {
        combine_f32_kernel<false><<<grid, 128, 0, s>>>(static_cast<const float4*>(yp), row_gate, token_rows, k_t, out, p.d, W, amax);
    } else if (p.dtype == DSMOE_BF16) {
        if (p.out_fp32)
            combine_bf16_kernel<true><<<grid, 128, 0, s>>>(static_cast<const uint4*>(yp), row_gate, token_rows, k_t, out,
                                                         p.d, W, amax);
        else
            combine_bf16_kernel<false><<<grid, 128, 0, s>>>(static_cast<const uint4*>(yp), row_gate, token_rows, k_t, out,
                                                          p.d, W, amax);
    } else {
        combine_f32_kernel<false><<<grid, 128, 0, s>>>(static_cast<const float4*>(yp), row_gate, token_rows, k_t, out, p.d, W, amax);
    }
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

// Selection statistics.  One warp per token; integer atomics only, so the counts do not depend on the order.
__global__ void __launch_bounds__(256) stats_kernel(const float* __restrict__ scores, const uint64_t* __restrict__ mask,
                                                    dsmoe_selection_stats* __restrict__ st, int T, int E, int mode, float eps,
                                                    int eps_normalized) {
    __shared__ int cnt_s[kMaxExperts];
    __shared__ unsigned long long near_s, a_s;
    __shared__ int zero_s;
    if (threadIdx.x < kMaxExperts) cnt_s[threadIdx.x] = 0;
    if (threadIdx.x == 0) {
        near_s = 0ull;
        a_s = 0ull;
        zero_s = 0;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const bool thr = mode == DSMOE_SELECT_THRESHOLD || mode == DSMOE_SELECT_THRESHOLD_TOPK;
    for (int t = blockIdx.x * 8 + (threadIdx.x >> 5); t < T; t += gridDim.x * 8) {
        const uint64_t m = mask[t];
        if (lane == 0) {
            atomicAdd(&a_s, (unsigned long long)__popcll(m));
            if (m == 0) atomicAdd(&zero_s, 1);
        }
        for (int e = lane; e < E; e += 32) {
            if ((m >> e) & 1ull) atomicAdd(&cnt_s[e], 1);
            if (thr) {
                const float sc = scores[(size_t)t * E + e];
                const float v = eps_normalized ? __fmul_rn(sc, (float)E) : sc;   // the value the rule compares
                if (fabs((double)v - (double)eps) <= 1e-6) atomicAdd(&near_s, 1ull);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < E && cnt_s[threadIdx.x]) atomicAdd(&st->counts[threadIdx.x], cnt_s[threadIdx.x]);
    if (threadIdx.x == 0) {
        atomicAdd(reinterpret_cast<unsigned long long*>(&st->assignments), a_s);
        atomicAdd(reinterpret_cast<unsigned long long*>(&st->near_threshold), near_s);
        atomicAdd(&st->zero_tokens, zero_s);
    }
}

__global__ void stats_finish_kernel(dsmoe_selection_stats* st, int E) {
    int n = 0;
    for (int e = 0; e < E; ++e) n += st->counts[e] == 0;
    st->empty_experts = n;
}

dsmoe_status launch_stats(const dsmoe_layer_desc& p, const float* scores, const uint64_t* mask,
                          dsmoe_selection_stats* stats, cudaStream_t s) {
    DSMOE_CUDA_TRY(cudaMemsetAsync(stats, 0, sizeof(dsmoe_selection_stats), s));
    if (p.T > 0) {
        const int grid = ceil_div(p.T, 8) < 1184 ? ceil_div(p.T, 8) : 1184;
        stats_kernel<<<grid, 256, 0, s>>>(scores, mask, stats, p.T, p.E, p.mode, p.eps, p.eps_normalized);
        DSMOE_CUDA_TRY(cudaGetLastError());
    }
    stats_finish_kernel<<<1, 1, 0, s>>>(stats, p.E);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_pack(const dsmoe_layer_desc& p, const void* W1, const void* W2, void* packed, cudaStream_t s) {
    const __nv_bfloat16* w1 = static_cast<const __nv_bfloat16*>(W1);
    const __nv_bfloat16* w2 = static_cast<const __nv_bfloat16*>(W2);
    __nv_bfloat16* w1t = static_cast<__nv_bfloat16*>(packed);
    __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    // W1[e]: [d,H] -> [d/64][H][64];  W2[e]: [H,d] -> [H/64][d][64]
    transpose_bf16_kernel<<<dim3(ceil_div(p.H, 32), ceil_div(p.d, 32), p.E), 256, 0, s>>>(w1, w1t, p.d, p.H);
    DSMOE_CUDA_TRY(cudaGetLastError());
    transpose_bf16_kernel<<<dim3(ceil_div(p.d, 32), ceil_div(p.H, 32), p.E), 256, 0, s>>>(w2, w2t, p.H, p.d);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace dsmoe
