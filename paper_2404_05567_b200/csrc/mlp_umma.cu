// Expert MLPs (Eq. 1's e(X) = GeLU(X.W1).W2) on the 5th-generation tensor cores: a persistent,
// warp-specialised GEMM whose operands arrive by TMA into 128-byte-swizzled shared memory, whose
// products are issued by one thread with tcgen05.mma into TMEM accumulators, and whose epilogue
// (GeLU, router gate, rounding) reads TMEM back with tcgen05.ld while the next tile's mainloop runs
// on the other half of TMEM.
//
//   warp 0      TMA producer         (one lane)
//   warp 1      MMA issuer           (one lane); owns the TMEM allocation
//   warps 2..5  epilogue             (warp w reads TMEM lanes 32*(w%4) .. +31)
//
// Three tilings share the kernel:
//   GROUPED     rows sorted by expert (sparse inference): tile = (expert, 128 rows, <=256 columns)
//   DENSE_UP    every expert on every token (dense forward): h[t, e*H + j] = S[t,e] * GeLU(x[t].W1[e][:,j])
//   DENSE_DOWN  out[t,:] = sum over (e,j) of that h times W2[e][j,:] -- the router-weighted sum of
//               Eq. 1 folded into the reduction dimension, so no grouping and no aggregation pass
#include "common.cuh"
#include "umma.cuh"

namespace dsmoe {

namespace {

constexpr int BM = 128, BK = 64, BN = 256, STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int B_STAGE_BYTES = BN * BK * 2;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 1024;

enum { GEMM_GROUPED = 0, GEMM_DENSE_UP = 1, GEMM_DENSE_DOWN = 2 };
enum { EPI_GELU = 0, EPI_STORE = 1 };

struct GemmParams {
    int mode, epi;
    int E;
    int n_per_expert;        // output columns per expert: H (up-projection) or d (down-projection)
    int k_per_expert;        // reduction length per expert: d (up) or H (down)
    int rows;                // rows of A: T (dense) or Amax (grouped)
    const int32_t* offsets;  // grouped: expert segments
    const float* gate;       // dense up: scores [T,E]; else null
    void* out;
    long long ld_out;        // elements
    int out_f32;
    int32_t* dev_status;
};

struct Tile {
    int row0, rows_valid, e, n0, bn, nk, out_col0;
};

struct Shared {
    uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    int bad_offsets;
    int tile_prefix[kMaxExperts + 1];
    int seg0[kMaxExperts], seg1[kMaxExperts];
};

__device__ __forceinline__ int total_tiles(const GemmParams& P, const Shared& sh) {
    const int ntn = (P.n_per_expert + BN - 1) / BN;
    if (P.mode == GEMM_GROUPED) return sh.tile_prefix[P.E];
    const int mt = (P.rows + BM - 1) / BM;
    return P.mode == GEMM_DENSE_UP ? mt * ntn * P.E : mt * ntn;
}

__device__ __forceinline__ Tile decode_tile(const GemmParams& P, const Shared& sh, int id) {
    Tile t;
    const int kbpe = P.k_per_expert / BK;
    if (P.mode == GEMM_GROUPED) {
        int e = 0;
        while (e + 1 < P.E && id >= sh.tile_prefix[e + 1]) ++e;
        const int local = id - sh.tile_prefix[e];
        const int cnt = sh.seg1[e] - sh.seg0[e];
        const int mtiles = (cnt + BM - 1) / BM;
        const int nt = local / mtiles, mt = local % mtiles;
        t.e = e;
        t.row0 = sh.seg0[e] + mt * BM;
        t.rows_valid = min(BM, sh.seg1[e] - t.row0);
        t.n0 = nt * BN;
        t.nk = kbpe;
        t.out_col0 = t.n0;
    } else {
        const int mtiles = (P.rows + BM - 1) / BM;
        const int ntn = (P.n_per_expert + BN - 1) / BN;
        const int mt = id % mtiles, rest = id / mtiles;
        t.row0 = mt * BM;
        t.rows_valid = min(BM, P.rows - t.row0);
        if (P.mode == GEMM_DENSE_UP) {
            t.e = rest / ntn;
            t.n0 = (rest % ntn) * BN;
            t.nk = kbpe;
            t.out_col0 = t.e * P.n_per_expert + t.n0;
        } else {
            t.e = 0;
            t.n0 = rest * BN;
            t.nk = kbpe * P.E;
            t.out_col0 = t.n0;
        }
    }
    t.bn = min(BN, P.n_per_expert - t.n0);
    return t;
}

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f)); }

__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;             // 128-byte swizzle wants 1024-byte aligned tiles
    const uint32_t smA = base, smB = base + STAGES * A_STAGE_BYTES;
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw + (base - raw) + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_u32(&sh.tfull[a]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.tempty[a]), 4);
        }
        sh.abort_flag = 0;
        sh.bad_offsets = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (P.mode == GEMM_GROUPED && threadIdx.x < P.E) {
        // segments as given, clamped so that a corrupt offsets array cannot send a tile out of range
        const int e = threadIdx.x;
        int s0 = P.offsets[e], s1 = P.offsets[e + 1];
        if (s0 < 0 || s1 < s0 || s1 > P.rows) {
            sh.bad_offsets = 1;
            s0 = s1 = 0;
        }
        sh.seg0[e] = s0;
        sh.seg1[e] = s1;
    }
    __syncthreads();
    if (P.mode == GEMM_GROUPED && threadIdx.x == 0) {
        const int ntn = (P.n_per_expert + BN - 1) / BN;
        int run = 0;
        for (int e = 0; e < P.E; ++e) {
            sh.tile_prefix[e] = run;
            run += ((sh.seg1[e] - sh.seg0[e] + BM - 1) / BM) * ntn;
        }
        sh.tile_prefix[P.E] = run;
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;
    const int ntiles = total_tiles(P, sh);
    const int kbpe = P.k_per_expert / BK;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool alive = true;
            for (int id = blockIdx.x; id < ntiles && alive; id += gridDim.x) {
                const Tile t = decode_tile(P, sh, id);
                for (int i = 0; i < t.nk; ++i) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                    ptx::mbar_expect_tx(bar, A_STAGE_BYTES + B_STAGE_BYTES);
                    int a_col, b_e, b_k;
                    if (P.mode == GEMM_DENSE_DOWN) {
                        b_e = i / kbpe;
                        b_k = (i % kbpe) * BK;
                        a_col = b_e * P.k_per_expert + b_k;
                    } else {
                        b_e = t.e;
                        b_k = i * BK;
                        a_col = b_k;
                    }
                    ptx::tma_load_2d(smA + s * A_STAGE_BYTES, &tmA, bar, a_col, t.row0);
                    ptx::tma_load_3d(smB + s * B_STAGE_BYTES, &tmB, bar, b_k, t.n0, b_e);
                    if (++s == STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!alive) {
                // copies already issued still land in this CTA's shared memory: give them time
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 200000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0, acc = 0;
            uint32_t ph = 0, aph = 0;
            bool alive = true;
            for (int id = blockIdx.x; id < ntiles && alive; id += gridDim.x) {
                const Tile t = decode_tile(P, sh, id);
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.tempty[acc]), aph ^ 1u, &sh.abort_flag)) break;
                ptx::tc_fence_after();
                const uint32_t idesc = ptx::make_idesc_bf16(BM, (uint32_t)t.bn);
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int i = 0; i < t.nk; ++i) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a0 = smA + s * A_STAGE_BYTES, b0 = smB + s * B_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        ptx::umma_bf16(d_tmem, ptx::make_desc_k_sw128(a0 + k * 32), ptx::make_desc_k_sw128(b0 + k * 32),
                                       idesc, (uint32_t)((i | k) != 0));
                    ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));   // slot reusable once these MMAs have read it
                    if (++s == STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (!alive) break;
                ptx::umma_commit(ptx::smem_u32(&sh.tfull[acc]));      // accumulator complete
                if (++acc == 2) {
                    acc = 0;
                    aph ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (4 warps)
        const int q = warp & 3;
        int acc = 0;
        uint32_t aph = 0;
        for (int id = blockIdx.x; id < ntiles; id += gridDim.x) {
            const Tile t = decode_tile(P, sh, id);
            if (!ptx::mbar_wait(ptx::smem_u32(&sh.tfull[acc]), aph, &sh.abort_flag)) break;
            ptx::tc_fence_after();
            const int row = q * 32 + lane;
            const bool valid = row < t.rows_valid;
            const long long grow = (long long)t.row0 + row;
            float g = 1.f;
            if (P.gate && valid) g = P.gate[grow * P.E + t.e];
            const uint32_t taddr = tmem_base + (uint32_t)(acc * BN) + ((uint32_t)(q * 32) << 16);
            for (int c = 0; c < t.bn; c += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(taddr + (uint32_t)c, r);
                ptx::tmem_ld_wait();
                if (valid) {
                    const long long o = grow * P.ld_out + t.out_col0 + c;
                    if (P.epi == EPI_GELU) {
                        uint4 pk[4];
                        __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            hv[j] = __floats2bfloat162_rn(g * gelu_erf(__uint_as_float(r[2 * j])),
                                                          g * gelu_erf(__uint_as_float(r[2 * j + 1])));
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + o);
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[j] = pk[j];
                    } else if (P.out_f32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(P.out) + o);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                 __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                    } else {
                        uint4 pk[4];
                        __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            hv[j] = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + o);
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[j] = pk[j];
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.tempty[acc]));
            if (++acc == 2) {
                acc = 0;
                aph ^= 1u;
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && P.dev_status) {
        if (sh.abort_flag) *P.dev_status = DSMOE_ERR_TIMEOUT;
        else if (sh.bad_offsets) *P.dev_status = DSMOE_ERR_INVALID_ARG;
    }
}

// ---------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 [rows, cols] row-major, box {64 cols, box_rows}, 128-byte swizzle
dsmoe_status make_map_2d(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return DSMOE_ERR_CUDA;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t es[2] = {1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSMOE_OK : DSMOE_ERR_CUDA;
}

// bf16 [E, n, k] row-major, box {64 k, box_n, 1}, 128-byte swizzle
dsmoe_status make_map_3d(CUtensorMap* m, const void* ptr, uint64_t E, uint64_t n, uint64_t k, uint32_t box_n) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return DSMOE_ERR_CUDA;
    const cuuint64_t dims[3] = {k, n, E};
    const cuuint64_t strides[2] = {k * 2, n * k * 2};
    const cuuint32_t box[3] = {BK, box_n, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSMOE_OK : DSMOE_ERR_CUDA;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

dsmoe_status launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmParams& P, int grid, cudaStream_t s) {
    static bool attr_set = false;
    if (!attr_set) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(umma_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
        attr_set = true;
    }
    umma_gemm_kernel<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(a, b, P);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace

bool umma_supported(const dsmoe_layer_desc& p) {
    return p.dtype == DSMOE_BF16 && (p.d % 64) == 0 && (p.H % 64) == 0;
}

dsmoe_status launch_mlp_umma(const dsmoe_layer_desc& p, const void* xp, const void* packed, const int32_t* offsets,
                             void* hbuf, void* yp, int32_t* dev_status, cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    if (!umma_supported(p)) return DSMOE_ERR_UNSUPPORTED;
    const size_t amax = amax_of(p);
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    CUtensorMap mA1, mB1, mA2, mB2;
    DSMOE_TRY(make_map_2d(&mA1, xp, amax, p.d, BM));
    DSMOE_TRY(make_map_3d(&mB1, w1t, p.E, p.H, p.d, BN));
    DSMOE_TRY(make_map_2d(&mA2, hbuf, amax, p.H, BM));
    DSMOE_TRY(make_map_3d(&mB2, w2t, p.E, p.d, p.H, BN));
    GemmParams up{GEMM_GROUPED, EPI_GELU, p.E, p.H, p.d, (int)amax, offsets, nullptr, hbuf, p.H, 0, dev_status};
    GemmParams down{GEMM_GROUPED, EPI_STORE, p.E, p.d, p.H, (int)amax, offsets, nullptr, yp, p.d, 0, dev_status};
    DSMOE_TRY(launch_gemm(mA1, mB1, up, sm_count(), s));
    DSMOE_TRY(launch_gemm(mA2, mB2, down, sm_count(), s));
    return DSMOE_OK;
}

dsmoe_status launch_layer_umma(const dsmoe_layer_desc& p, const void* x, const void* packed, const float* scores,
                               const uint64_t* mask, const int32_t* k_t, int32_t* counts_out, void* out, char* ws,
                               const WsLayout& L, int32_t* dev_status, cudaStream_t s, bool* done) {
    *done = false;
    if (!umma_supported(p) || p.mode != DSMOE_SELECT_ALL) return DSMOE_OK;
    // Dense forward: gate folded into h, aggregation folded into the down-projection's reduction.
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    void* hg = ws + L.h;                                        // [T, E*H] bf16
    CUtensorMap mA1, mB1, mA2, mB2;
    DSMOE_TRY(make_map_2d(&mA1, x, p.T, p.d, BM));
    DSMOE_TRY(make_map_3d(&mB1, w1t, p.E, p.H, p.d, BN));
    DSMOE_TRY(make_map_2d(&mA2, hg, p.T, (uint64_t)p.E * p.H, BM));
    DSMOE_TRY(make_map_3d(&mB2, w2t, p.E, p.d, p.H, BN));
    const int out_f32 = p.out_fp32 ? 1 : 0;
    GemmParams up{GEMM_DENSE_UP, EPI_GELU, p.E, p.H, p.d, p.T, nullptr, scores, hg, (long long)p.E * p.H, 0, dev_status};
    GemmParams down{GEMM_DENSE_DOWN, EPI_STORE, p.E, p.d, p.H, p.T, nullptr, nullptr, out, p.d, out_f32, dev_status};
    const int mt = ceil_div(p.T, BM);
    const int tiles_up = mt * ceil_div(p.H, BN) * p.E, tiles_down = mt * ceil_div(p.d, BN);
    DSMOE_TRY(launch_gemm(mA1, mB1, up, tiles_up < sm_count() ? tiles_up : sm_count(), s));
    DSMOE_TRY(launch_gemm(mA2, mB2, down, tiles_down < sm_count() ? tiles_down : sm_count(), s));
    if (counts_out) {
        int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
        int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
        DSMOE_TRY(launch_finalize(p, mask, counts, offsets, reinterpret_cast<int32_t*>(ws + L.chunk_prefix), counts_out, s));
    }
    (void)k_t;
    *done = true;
    return DSMOE_OK;
}

}  // namespace dsmoe
