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
//   SMALL_UP / SMALL_DOWN   the same two products for a handful of tokens (decode), where time is
//               the reading of the selected experts' weights: only experts that some token selected
//               are streamed, each weight byte once, in contiguous slabs split evenly over the
//               CTAs (16 weight rows for the up-projection, one 64-wide reduction block for the
//               down-projection, whose partial sums a short fix-up kernel adds in a fixed order)
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

enum { GEMM_GROUPED = 0, GEMM_DENSE_UP = 1, GEMM_DENSE_DOWN = 2, GEMM_SMALL_UP = 3, GEMM_SMALL_DOWN = 4 };
enum { EPI_GELU = 0, EPI_STORE = 1, EPI_PARTIAL = 2 };
constexpr int kUpUnit = 16;          // weight rows per work unit of SMALL_UP

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
    const uint64_t* mask;    // small-T modes: selection words of the T tokens
    int a_box_rows;          // rows per TMA box of A (128, or T rounded up to 8 in the small-T modes)
    int b_box_rows;          // rows per TMA box of B (256, or 16 in SMALL_UP)
};

struct Tile {
    int row0, rows_valid, e, n0, bn, nk, out_col0;
    int kstart, seg;         // SMALL_DOWN: first global reduction block, partial-sum slot
};

struct Shared {
    uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    int bad_offsets;
    int tile_prefix[kMaxExperts + 1];
    int seg0[kMaxExperts], seg1[kMaxExperts];
    unsigned long long active_mask;   // small-T modes: experts selected by at least one token
    int n_act;
    int active[kMaxExperts];
};

// Walks the tiles of one CTA.  The large-T tilings stride a global tile index over the grid; the
// small-T tilings cut this CTA's contiguous range of work units into tiles.
struct TileIter {
    int id, u0, u1, r_first;

    __device__ __forceinline__ void init(const GemmParams& P, const Shared& sh) {
        id = blockIdx.x;
        if (P.mode == GEMM_SMALL_UP || P.mode == GEMM_SMALL_DOWN) {
            const int kbpe = P.k_per_expert / BK;
            const int total = P.mode == GEMM_SMALL_UP
                                  ? sh.n_act * (P.n_per_expert / kUpUnit)
                                  : ((P.n_per_expert + BN - 1) / BN) * sh.n_act * kbpe;
            const int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
            u0 = min(total, (int)blockIdx.x * per);
            u1 = min(total, u0 + per);
            const int U = sh.n_act * kbpe;
            r_first = (P.mode == GEMM_SMALL_DOWN && U > 0) ? u0 / U : 0;
        }
    }

    __device__ __forceinline__ bool next(const GemmParams& P, const Shared& sh, Tile& t);
};

__device__ __forceinline__ int total_tiles(const GemmParams& P, const Shared& sh) {
    const int ntn = (P.n_per_expert + BN - 1) / BN;
    if (P.mode == GEMM_GROUPED) return sh.tile_prefix[P.E];
    const int mt = (P.rows + BM - 1) / BM;
    return P.mode == GEMM_DENSE_UP ? mt * ntn * P.E : mt * ntn;
}

__device__ __forceinline__ bool TileIter::next(const GemmParams& P, const Shared& sh, Tile& t) {
    const int kbpe = P.k_per_expert / BK;
    t.kstart = 0;
    t.seg = 0;
    if (P.mode == GEMM_SMALL_UP) {
        // units of 16 weight rows over the selected experts, concatenated; a tile stays inside one expert
        if (u0 >= u1) return false;
        const int upe = P.n_per_expert / kUpUnit;
        const int ei = u0 / upe, in_e = u0 % upe;
        const int len = min(min(u1 - u0, upe - in_e), BN / kUpUnit);
        t.e = sh.active[ei];
        t.row0 = 0;
        t.rows_valid = P.rows;
        t.n0 = in_e * kUpUnit;
        t.bn = len * kUpUnit;
        t.nk = kbpe;
        t.out_col0 = t.e * P.n_per_expert + t.n0;
        u0 += len;
        return true;
    }
    if (P.mode == GEMM_SMALL_DOWN) {
        // units = (256-column range, selected expert, 64-wide reduction block); a tile stays inside one range
        if (u0 >= u1) return false;
        const int U = sh.n_act * kbpe;
        const int r = u0 / U, start = u0 % U;
        const int len = min(u1 - u0, U - start);
        t.e = 0;
        t.row0 = 0;
        t.rows_valid = P.rows;
        t.n0 = r * BN;
        t.bn = min(BN, P.n_per_expert - t.n0);
        t.nk = len;
        t.kstart = start;
        t.seg = r - r_first;
        t.out_col0 = 0;
        u0 += len;
        return true;
    }
    if (id >= total_tiles(P, sh)) return false;
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
    id += gridDim.x;
    return true;
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
    const bool small = P.mode == GEMM_SMALL_UP || P.mode == GEMM_SMALL_DOWN;

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
        sh.active_mask = 0ull;
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
    if (small && threadIdx.x < P.rows) atomicOr(&sh.active_mask, (unsigned long long)P.mask[threadIdx.x]);
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
    if (small && threadIdx.x == 0) {
        unsigned long long m = sh.active_mask;
        if (P.E < 64) m &= (1ull << P.E) - 1ull;
        int n = 0;
        for (int e = 0; e < P.E; ++e)
            if ((m >> e) & 1ull) sh.active[n++] = e;
        sh.n_act = n;
    }
    if (small) __syncthreads();
    const uint32_t tmem_base = sh.tmem_base;
    const int kbpe = P.k_per_expert / BK;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool alive = true;
            const uint32_t a_bytes = (uint32_t)P.a_box_rows * BK * 2;
            TileIter it;
            it.init(P, sh);
            Tile t;
            while (alive && it.next(P, sh, t)) {
                const int b_boxes = (t.bn + P.b_box_rows - 1) / P.b_box_rows;
                const uint32_t b_box_bytes = (uint32_t)P.b_box_rows * BK * 2;
                for (int i = 0; i < t.nk; ++i) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                    ptx::mbar_expect_tx(bar, a_bytes + b_boxes * b_box_bytes);
                    int a_col, b_e, b_k;
                    if (P.mode == GEMM_DENSE_DOWN || P.mode == GEMM_SMALL_DOWN) {
                        const int g = t.kstart + i;
                        const int ei = g / kbpe;
                        b_e = P.mode == GEMM_SMALL_DOWN ? sh.active[ei] : ei;
                        b_k = (g % kbpe) * BK;
                        a_col = b_e * P.k_per_expert + b_k;
                    } else {
                        b_e = t.e;
                        b_k = i * BK;
                        a_col = b_k;
                    }
                    ptx::tma_load_2d(smA + s * A_STAGE_BYTES, &tmA, bar, a_col, t.row0);
                    for (int b = 0; b < b_boxes; ++b)
                        ptx::tma_load_3d(smB + s * B_STAGE_BYTES + b * b_box_bytes, &tmB, bar, b_k,
                                         t.n0 + b * P.b_box_rows, b_e);
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
            TileIter it;
            it.init(P, sh);
            Tile t;
            while (alive && it.next(P, sh, t)) {
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
        TileIter it;
        it.init(P, sh);
        Tile t;
        while (it.next(P, sh, t)) {
            if (!ptx::mbar_wait(ptx::smem_u32(&sh.tfull[acc]), aph, &sh.abort_flag)) break;
            ptx::tc_fence_after();
            const int row = q * 32 + lane;
            const bool valid = row < t.rows_valid;
            const long long grow = (long long)t.row0 + row;
            float g = 1.f;
            if (P.gate && valid) {
                g = P.gate[grow * P.E + t.e];
                if (small && !((P.mask[grow] >> t.e) & 1ull)) g = 0.f;   // expert not selected by this token
            }
            const uint32_t taddr = tmem_base + (uint32_t)(acc * BN) + ((uint32_t)(q * 32) << 16);
            // warps whose 32 TMEM lanes hold no valid row skip the read-back altogether
            const bool warp_has_rows = q * 32 < t.rows_valid;
            for (int c = 0; warp_has_rows && c < t.bn; c += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(taddr + (uint32_t)c, r);
                ptx::tmem_ld_wait();
                if (!valid) continue;
                const int ncol = min(32, t.bn - c);   // 16 or 32 (bn is a multiple of 16)
                if (P.epi == EPI_GELU) {
                    const long long o = grow * P.ld_out + t.out_col0 + c;
                    uint4 pk[4];
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        hv[j] = __floats2bfloat162_rn(g * gelu_erf(__uint_as_float(r[2 * j])),
                                                      g * gelu_erf(__uint_as_float(r[2 * j + 1])));
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + o);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j * 8 < ncol) dst[j] = pk[j];
                } else if (P.epi == EPI_PARTIAL) {
                    // fp32 partial sums of this CTA's share of the reduction: slot (cta, seg), row, 256 columns
                    float* dstf = static_cast<float*>(P.out) +
                                  (((long long)blockIdx.x * 2 + t.seg) * P.rows + grow) * BN + c;
                    float4* dst = reinterpret_cast<float4*>(dstf);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j * 4 < ncol)
                            dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                 __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                } else if (P.out_f32) {
                    const long long o = grow * P.ld_out + t.out_col0 + c;
                    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(P.out) + o);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j * 4 < ncol)
                            dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                 __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                } else {
                    const long long o = grow * P.ld_out + t.out_col0 + c;
                    uint4 pk[4];
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        hv[j] = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + o);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j * 8 < ncol) dst[j] = pk[j];
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

// Adds the partial sums of SMALL_DOWN in a fixed order (ascending CTA) and writes out[T,d].
// Grid (column ranges of 256, T); the partition arithmetic mirrors TileIter::init / next.
__global__ void __launch_bounds__(BN) small_fixup_kernel(const float* __restrict__ partial, const uint64_t* __restrict__ mask,
                                                         void* __restrict__ out, int T, int d, int E, int kbpe, int G,
                                                         int out_f32) {
    __shared__ unsigned long long act;
    if (threadIdx.x == 0) act = 0ull;
    __syncthreads();
    if (threadIdx.x < T) atomicOr(&act, (unsigned long long)mask[threadIdx.x]);
    __syncthreads();
    unsigned long long m = act;
    if (E < 64) m &= (1ull << E) - 1ull;
    const int U = __popcll(m) * kbpe;
    const int r = blockIdx.x, t = blockIdx.y;
    const int c = r * BN + threadIdx.x;
    if (c >= d) return;
    float sum = 0.f;
    if (U > 0) {
        const int nr = (d + BN - 1) / BN;
        const int total = nr * U;
        const int per = (total + G - 1) / G;
        const int i0 = (r * U) / per, i1 = ((r + 1) * U - 1) / per;
        for (int i = i0; i <= i1; ++i) {
            const int seg = r - (i * per) / U;
            sum += partial[(((long long)i * 2 + seg) * T + t) * BN + threadIdx.x];
        }
    }
    if (out_f32) static_cast<float*>(out)[(long long)t * d + c] = sum;
    else static_cast<__nv_bfloat16*>(out)[(long long)t * d + c] = __float2bfloat16_rn(sum);
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

// Optional per-launch timing of the expert GEMMs (a measurement aid for benchmarks): event pairs
// around each launch of the most recent call.
constexpr int kMaxTimed = 8;
struct Timing {
    bool on = false, made = false;
    int n = 0;
    cudaEvent_t start[kMaxTimed], stop[kMaxTimed];
} g_timing;

dsmoe_status launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmParams& P, int grid, cudaStream_t s) {
    static bool attr_set = false;
    if (!attr_set) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(umma_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
        attr_set = true;
    }
    const bool timed = g_timing.on && g_timing.n < kMaxTimed;
    if (timed) DSMOE_CUDA_TRY(cudaEventRecord(g_timing.start[g_timing.n], s));
    umma_gemm_kernel<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(a, b, P);
    DSMOE_CUDA_TRY(cudaGetLastError());
    if (timed) DSMOE_CUDA_TRY(cudaEventRecord(g_timing.stop[g_timing.n++], s));
    return DSMOE_OK;
}

}  // namespace

void timing_reset() { g_timing.n = 0; }

dsmoe_status timing_enable(int on) {
    if (on && !g_timing.made) {
        for (int i = 0; i < kMaxTimed; ++i) {
            DSMOE_CUDA_TRY(cudaEventCreate(&g_timing.start[i]));
            DSMOE_CUDA_TRY(cudaEventCreate(&g_timing.stop[i]));
        }
        g_timing.made = true;
    }
    g_timing.on = on != 0;
    g_timing.n = 0;
    return DSMOE_OK;
}

dsmoe_status timing_last(float* ms, int n_max, int* n) {
    *n = 0;
    if (!g_timing.on) return DSMOE_OK;
    for (int i = 0; i < g_timing.n && i < n_max; ++i) {
        DSMOE_CUDA_TRY(cudaEventSynchronize(g_timing.stop[i]));
        DSMOE_CUDA_TRY(cudaEventElapsedTime(&ms[i], g_timing.start[i], g_timing.stop[i]));
        *n = i + 1;
    }
    return DSMOE_OK;
}

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
    GemmParams up{GEMM_GROUPED, EPI_GELU, p.E, p.H, p.d, (int)amax, offsets, nullptr, hbuf, p.H, 0, dev_status,
                  nullptr, BM, BN};
    GemmParams down{GEMM_GROUPED, EPI_STORE, p.E, p.d, p.H, (int)amax, offsets, nullptr, yp, p.d, 0, dev_status,
                    nullptr, BM, BN};
    DSMOE_TRY(launch_gemm(mA1, mB1, up, sm_count(), s));
    DSMOE_TRY(launch_gemm(mA2, mB2, down, sm_count(), s));
    return DSMOE_OK;
}

// Few tokens (decode): every token rides in one 128-row tile, only the selected experts' weights are
// streamed, and the router gate (zero for an unselected pair) is folded into h, so the layer needs no
// grouping and no aggregation pass.
static dsmoe_status launch_layer_small(const dsmoe_layer_desc& p, const void* x, const void* packed,
                                       const float* scores, const uint64_t* mask, void* out, char* ws,
                                       const WsLayout& L, int32_t* dev_status, cudaStream_t s) {
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    void* hg = ws + L.h;                                        // [T, E*H] bf16
    float* partial = reinterpret_cast<float*>(ws + L.partial);
    const int t_pad = (p.T + 7) / 8 * 8;
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    CUtensorMap mA1, mB1, mA2, mB2;
    DSMOE_TRY(make_map_2d(&mA1, x, p.T, p.d, t_pad));
    DSMOE_TRY(make_map_3d(&mB1, w1t, p.E, p.H, p.d, kUpUnit));
    DSMOE_TRY(make_map_2d(&mA2, hg, p.T, (uint64_t)p.E * p.H, t_pad));
    DSMOE_TRY(make_map_3d(&mB2, w2t, p.E, p.d, p.H, BN));
    GemmParams up{GEMM_SMALL_UP, EPI_GELU, p.E, p.H, p.d, p.T, nullptr, scores, hg, (long long)p.E * p.H, 0,
                  dev_status, mask, t_pad, kUpUnit};
    GemmParams down{GEMM_SMALL_DOWN, EPI_PARTIAL, p.E, p.d, p.H, p.T, nullptr, nullptr, partial, BN, 1,
                    dev_status, mask, t_pad, BN};
    DSMOE_TRY(launch_gemm(mA1, mB1, up, G, s));
    DSMOE_TRY(launch_gemm(mA2, mB2, down, G, s));
    small_fixup_kernel<<<dim3(ceil_div(p.d, BN), p.T), BN, 0, s>>>(partial, mask, out, p.T, p.d, p.E, p.H / BK, G,
                                                                  (p.out_fp32 || p.dtype == DSMOE_F32) ? 1 : 0);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

dsmoe_status launch_layer_umma(const dsmoe_layer_desc& p, const void* x, const void* packed, const float* scores,
                               const uint64_t* mask, const int32_t* k_t, int32_t* counts_out, void* out, char* ws,
                               const WsLayout& L, int32_t* dev_status, cudaStream_t s, bool* done) {
    *done = false;
    (void)k_t;
    if (!umma_supported(p)) return DSMOE_OK;
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    if (p.T <= kSmallMaxT && ceil_div(p.d, BN) <= G) {
        DSMOE_TRY(launch_layer_small(p, x, packed, scores, mask, out, ws, L, dev_status, s));
    } else if (p.mode == DSMOE_SELECT_ALL) {
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
        GemmParams up{GEMM_DENSE_UP, EPI_GELU, p.E, p.H, p.d, p.T, nullptr, scores, hg, (long long)p.E * p.H, 0,
                      dev_status, nullptr, BM, BN};
        GemmParams down{GEMM_DENSE_DOWN, EPI_STORE, p.E, p.d, p.H, p.T, nullptr, nullptr, out, p.d, out_f32,
                        dev_status, nullptr, BM, BN};
        const int mt = ceil_div(p.T, BM);
        const int tiles_up = mt * ceil_div(p.H, BN) * p.E, tiles_down = mt * ceil_div(p.d, BN);
        DSMOE_TRY(launch_gemm(mA1, mB1, up, tiles_up < sm_count() ? tiles_up : sm_count(), s));
        DSMOE_TRY(launch_gemm(mA2, mB2, down, tiles_down < sm_count() ? tiles_down : sm_count(), s));
    } else {
        return DSMOE_OK;
    }
    if (counts_out) {
        int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
        int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
        DSMOE_TRY(launch_finalize(p, mask, counts, offsets, reinterpret_cast<int32_t*>(ws + L.chunk_prefix), counts_out, s));
    }
    *done = true;
    return DSMOE_OK;
}

}  // namespace dsmoe
