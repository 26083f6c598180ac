// The whole layer (Eq. 1) for a handful of tokens -- a decoding step with up to 8 sequences -- in one cooperative
// launch in which a CTA never waits for another one between the two projections.
//
// With so few tokens the layer is bound by reading the selected experts' weights once, and the time is so short
// (100 MB at T = 1: 16 us at the memory's speed) that every hand-over between CTAs shows.  So the work is cut along
// the experts' hidden units: a CTA owns a contiguous run of 16-wide units of the selected experts' hidden layers and
// does everything that touches them,
//
//     router   every CTA computes the scores and the selection of every token itself (the same arithmetic in the
//              same order, hence the same result everywhere: nothing to agree on, no grid barrier)
//     up       a[k,t] = GeLU(W1[e][:,k] . x[t]) for its hidden units k: the weights are the M operand of the MMA
//              (128 hidden units per instruction), the tokens, padded to 16, its N operand
//     gate     hg[t,k] = [e in sel(t)] S[t,e] a[k,t] goes to SHARED memory as bf16, laid out as the next MMA's operand
//     down     partial[c,t] = sum over its k of W2[e][k,c] hg[t,k]: all d output columns as M tiles of 128 in TMEM,
//              the CTA's hidden units as the reduction, 16 at a time
//
// and only then meets the others: its fp32 partial output [T,d] goes to global memory, one grid barrier, and every
// CTA adds the partial outputs for its share of out[T,d] in a fixed order (bit-reproducible).  The hidden
// activations never leave the SM, and W1 and W2 are one uninterrupted stream through one ring of shared memory.
//
//   warp 0      TMA producer (one lane)          warp 1   MMA issuer (one lane); owns the TMEM allocation
//   warps 2..13 router, then the two epilogues (TMEM -> GeLU, gate -> shared memory; TMEM -> partial output), then the sum
//
// Every wait -- mbarrier, flag or grid barrier -- is bounded; on expiry the CTA sets an abort flag, every role leaves
// its loop, TMEM is freed and DSMOE_ERR_TIMEOUT is written to *dev_status.
#include "common.cuh"
#include "router_device.cuh"
#include "tensor_maps.cuh"
#include "umma.cuh"

namespace dsmoe {

namespace {

constexpr int FT_THREADS = 448;
constexpr int FT_EPI = FT_THREADS - 64;          // router / epilogue threads
constexpr int FT_N = 16;                         // token columns of every MMA
constexpr int FT_UNIT = 16;                      // hidden units per work unit = reduction length of one down-projection MMA
// The copy engine has only a few copies per SM under way at a time, whatever their size (about 4.5 per microsecond
// from HBM), so every copy is made as large as a ring slot: up to 32 KB, which four slots turn into the memory's
// full rate.  A narrow up-projection tile therefore brings several 64-wide blocks of d per copy, and a
// down-projection copy brings up to 1024 output columns of one hidden unit.  The tokens are not copied per slot at
// all: the router warps put them into shared memory once, as the MMA's N operand.
constexpr int FT_SLOT = 32 * 1024;
#ifndef DSMOE_FUSED_RING_SLOTS
#define DSMOE_FUSED_RING_SLOTS 4
#endif
constexpr int FT_STAGES = DSMOE_FUSED_RING_SLOTS;
constexpr int FT_RING = FT_STAGES * FT_SLOT;
constexpr int FT_XBLOCK = 8 * 128;               // one 64-wide block of the tokens in shared memory: 8 rows of 128 bytes
constexpr int FT_MAXTILES = 16;
constexpr int FT_HG_BYTES = kFusedMaxUnits * FT_N * 32;
constexpr int FT_TMEM_COLS = 512;
constexpr int FT_ROUTER_BATCH = 12;              // rows of Wr a router thread loads at once
constexpr int FT_FIX_BATCH = 16;
constexpr int FT_RED_FLOATS = FT_EPI;            // shared scratch of the final sum

struct FusedParams {
    int T, d, H, E;
    const __nv_bfloat16* x;
    const float* Wr;
    const float* br;
    SelParams sel;
    float* scores;
    uint64_t* mask;
    int32_t* k_t;
    int32_t* counts_out;     // nullable
    float* partial;          // [grid][T][d]
    void* out;
    int out_f32;
    int* sync;               // 8 ints, zero at launch: grid-barrier counters [0], [1] and an abort flag [4]
    int simt_up;             // up-projection on the CUDA cores (T <= 4) instead of the tensor cores
    int32_t* dev_status;
};

struct FShared {
    uint64_t full[FT_STAGES], empty[FT_STAGES];
    uint64_t d1_full, hg_ready, d2_full;
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int geo_ready;
    int n_act, u0, u1;                   // this CTA's units [u0, u1) of the n_act * H / 16 of the selected experts
    // ... cut at the expert boundaries into up-projection tiles of at most 8 units (128 hidden units, the MMA's M):
    // expert, first unit inside the expert, units, first unit counted from u0
    int ntiles, tile_e[FT_MAXTILES], tile_iu0[FT_MAXTILES], tile_len[FT_MAXTILES], tile_ul0[FT_MAXTILES];
    int nchain;                          // accumulators per tile (see the MMA issuer)
    int active[kMaxExperts];             // the selected experts, ascending
    uint64_t mask_s[kFusedMaxT];
    float score_s[kFusedMaxT][kMaxExperts];
#ifdef DSMOE_TRACE
    unsigned long long trace[32];
#endif
};
#ifdef DSMOE_TRACE
// Diagnostic build only (-DDSMOE_TRACE): per-CTA time stamps (globaltimer ns) of the kernel's milestones.
__device__ unsigned long long g_trace_fused[192][32];
#define TRACE(i) sh.trace[i] = ptx::globaltimer_ns()
#else
#define TRACE(i)
#endif
constexpr int FT_SHARED_BYTES = 4096;
static_assert(sizeof(FShared) <= FT_SHARED_BYTES, "FShared must fit its slot");
// ring | tokens (d / 64 + 1 blocks) | gated activations | FShared | scratch of the final sum
constexpr size_t ft_smem_bytes(int d) {
    return 1024 + (size_t)FT_RING + (size_t)(d / 64 + 1) * FT_XBLOCK + FT_HG_BYTES + FT_SHARED_BYTES + FT_RED_FLOATS * 4;
}
static_assert(ft_smem_bytes(4096) <= 227 * 1024, "shared memory of one CTA");
static_assert(kFusedMaxT * 16 * kMaxExperts * 4 <= FT_RING, "the router's scratch borrows the ring");

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f)); }

// first row of the tile (64 k of block kb, rows n0 ..) in the packed weights seen as [E][(K/64)*N][64]
__device__ __forceinline__ int wrow(int kb, int n0, int N) { return kb * N + n0; }

// Shared-memory operand descriptor for a K-major bf16 tile of 16 reduction elements: rows of 32 bytes written with
// the 32-byte swizzle (by TMA, or by hand in the same pattern), groups of 8 rows 256 bytes apart.
__device__ __forceinline__ uint64_t make_desc_k_sw32(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(256 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)6 << 61;                             // layout type: 32-byte swizzle
    return d;
}

__device__ __forceinline__ void grid_arrive(int* sync, int idx) {
    __threadfence();
    atomicAdd(sync + idx, 1);
}
__device__ __forceinline__ bool grid_wait(int* sync, int idx, int target, volatile int* abort_flag) {
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t spin = 0;; ++spin) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(sync + idx) : "memory");
        if (v >= target) return true;
        if ((spin & 0x3f) == 0x3f) {
            int ab;
            asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(ab) : "l"(sync + 4) : "memory");
            if (ab || *abort_flag || ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(sync + 4, 1);
                return false;
            }
        }
    }
}

// Bounded wait for the router's partition; false = gave up.
__device__ __forceinline__ bool wait_geo(FShared& sh) {
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t spin = 0;; ++spin) {
        if (sh.geo_ready) return true;
        if ((spin & 0xff) == 0xff) {
            if (sh.abort_flag) return false;
            if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
                sh.abort_flag = 1;
                return false;
            }
        }
    }
}

__global__ void __launch_bounds__(FT_THREADS, 1)
fused_decode_kernel(const __grid_constant__ BMapsUp tmW1, const __grid_constant__ BMapsDown tmW2, const FusedParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, T = P.T, E = P.E;
    const int upe = P.H / FT_UNIT;                       // units per expert
    const int nkb = P.d / 64;
    const uint32_t xs_bytes = (uint32_t)(nkb + 1) * FT_XBLOCK;
    const uint32_t ring = base, xs_addr = base + FT_RING, hg_addr = xs_addr + xs_bytes;
    uint8_t* xs = smem + FT_RING;
    uint8_t* hg = xs + xs_bytes;
    FShared& sh = *reinterpret_cast<FShared*>(hg + FT_HG_BYTES);
    float* red = reinterpret_cast<float*>(hg + FT_HG_BYTES + FT_SHARED_BYTES);

    if (threadIdx.x == 0) {
        for (int s = 0; s < FT_STAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&sh.d1_full), 1);
        ptx::mbar_init(ptx::smem_u32(&sh.hg_ready), 1);
        ptx::mbar_init(ptx::smem_u32(&sh.d2_full), 1);
        sh.abort_flag = 0;
        sh.geo_ready = 0;
#ifdef DSMOE_TRACE
        for (int i = 0; i < 32; ++i) sh.trace[i] = 0;
        TRACE(0);
#endif
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmW2.m);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), FT_TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0 && wait_geo(sh)) {
            const uint64_t wpol = ptx::policy_evict_first();    // weights are read once: first to leave L2
            const int u0 = sh.u0, nu = sh.u1 - sh.u0;
            int s = 0;
            uint32_t ph = 0;
            bool alive = true;
            TRACE(3);
            // up-projection: tile by tile, kbp reduction blocks per copy
            for (int ti = 0; alive && ti < sh.ntiles; ++ti) {
                const int len = sh.tile_len[ti], kbp = tmW1.kbp[len - 1];
                for (int g = 0; g * kbp < nkb; ++g) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                    ptx::mbar_expect_tx(bar, (uint32_t)(kbp * len * FT_UNIT * 128));     // blocks past d arrive as zeros
                    ptx::tma_load_4d_hint(ring + s * FT_SLOT, &tmW1.m[len - 1], bar, 0, sh.tile_iu0[ti] * FT_UNIT, g * kbp,
                                          sh.tile_e[ti], wpol);
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            TRACE(14);
            // down-projection: unit by unit, `ch` chunks of 256 output columns per copy
            const int nch = P.d / 256, ch = tmW2.ch;
            for (int j = 0; alive && j < nu; ++j) {
                const int u = u0 + j, e = sh.active[u / upe], hid = (u % upe) * FT_UNIT;
                for (int cg = 0; cg * ch < nch; ++cg) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                    ptx::mbar_expect_tx(bar, (uint32_t)(ch * 256 * 32));
                    ptx::tma_load_5d_hint(ring + s * FT_SLOT, &tmW2.m, bar, hid % 64, 0, cg * ch, hid / 64, e, wpol);
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            TRACE(15);
            if (!alive) {
                const uint64_t t0 = ptx::globaltimer_ns();   // copies already issued still land in this CTA's smem
                while (ptx::globaltimer_ns() - t0 < 200000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && wait_geo(sh)) {
            const int nu = sh.u1 - sh.u0;
            const uint32_t idesc = ptx::make_idesc_bf16(128, FT_N);
            int s = 0;
            uint32_t ph = 0;
            bool alive = nu > 0;
            // D1[tile][k, t] = sum over d of W1 rows (M) x tokens (N).  The M operand is read 128 rows deep whatever the
            // tile's height: what lies beyond it in shared memory only reaches TMEM lanes that nobody looks at.
            // Likewise the tokens' rows 8..15 (the next block's bytes).  These MMAs are tiny (128 x 16 x 16) and an
            // MMA waits for the previous one into the same accumulator, so a tile's reduction over d is spread over
            // `nchain` accumulators (64-wide block kb goes to accumulator kb % nchain, at TMEM columns
            // 16 (tile nchain + kb % nchain) ..), which the epilogue adds up.
            const int nchain = sh.nchain;
            for (int ti = 0; alive && !P.simt_up && ti < sh.ntiles; ++ti) {
                const int len = sh.tile_len[ti], kbp = tmW1.kbp[len - 1];
                for (int g = 0; g * kbp < nkb; ++g) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
#ifdef DSMOE_TRACE
                    if (sh.trace[4] == 0) TRACE(4);
#endif
                    const uint32_t slot = ring + s * FT_SLOT;
                    for (int kbi = 0; kbi < kbp && g * kbp + kbi < nkb; ++kbi) {
                        const int kb = g * kbp + kbi;
                        const uint32_t a0 = slot + kbi * len * (FT_UNIT * 128), b0 = xs_addr + kb * FT_XBLOCK;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            ptx::umma_bf16(tmem_base + (uint32_t)((ti * nchain + kb % nchain) * FT_N),
                                           ptx::make_desc_k_sw128(a0 + k * 32), ptx::make_desc_k_sw128(b0 + k * 32), idesc,
                                           (uint32_t)(kb >= nchain || k != 0));
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (P.simt_up) {
                // the CUDA cores took the up-projection's copies off the ring: the down-projection's follow them
                int n_up = 0;
                for (int ti = 0; ti < sh.ntiles; ++ti) {
                    const int kbp = tmW1.kbp[sh.tile_len[ti] - 1];
                    n_up += (nkb + kbp - 1) / kbp;
                }
                s = n_up % FT_STAGES;
                ph = (uint32_t)(n_up / FT_STAGES) & 1u;
            }
            TRACE(5);
            if (alive) {
                if (!P.simt_up) ptx::umma_commit(ptx::smem_u32(&sh.d1_full));
                // the gated activations in shared memory (and D1 read out of TMEM: D2 takes its place)
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.hg_ready), 0u, &sh.abort_flag)) alive = false;
                ptx::tc_fence_after();
            }
            // D2[c][col, t] += W2 rows of unit j (M = 128 output columns of chunk c, K = 16) x hg of unit j (N)
            const int nch = P.d / 256, ch = tmW2.ch;
            for (int j = 0; alive && j < nu; ++j) {
                for (int cg = 0; cg * ch < nch; ++cg) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t slot = ring + s * FT_SLOT;
                    for (int c = 0; c < 2 * ch && (cg * ch * 2 + c) * 128 < P.d; ++c)
                        ptx::umma_bf16(tmem_base + (uint32_t)((cg * ch * 2 + c) * FT_N), make_desc_k_sw32(slot + c * 4096),
                                       make_desc_k_sw32(hg_addr + j * (FT_N * 32)), idesc, (uint32_t)(j != 0));
                    ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            TRACE(8);
            if (alive) ptx::umma_commit(ptx::smem_u32(&sh.d2_full));
        }
    } else {
        // ------------------------------------------------------------ router, epilogues, final sum (12 warps)
        const int etid = (int)threadIdx.x - 64;
#define FT_SYNC() asm volatile("bar.sync 1, %0;" ::"n"(FT_EPI) : "memory")
        // ---- the tokens in shared memory.  For the tensor cores: the up-projection's N operand, per 64-wide block of d
        // 8 rows of 128 bytes in the 128-byte swizzle (16-byte piece c of row t sits at piece c ^ t), rows T.. zero.
        // For the CUDA cores (simt_up): fp32, per (block, token) the low halves of the eight 8-element pieces (16 bytes
        // each, 128 bytes in all), then the high halves, so that 8 lanes read them without bank conflicts.
        if (P.simt_up) {
            for (int i = etid; i < nkb * T * 8; i += FT_EPI) {
                const int c = i & 7, kt = i >> 3, kb = kt / T, t = kt % T;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(P.x + (size_t)t * P.d + kb * 64) + c);
                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
                const float2 a = __bfloat1622float2(h2[0]), b = __bfloat1622float2(h2[1]), cc = __bfloat1622float2(h2[2]),
                             dd = __bfloat1622float2(h2[3]);
                float4* dst = reinterpret_cast<float4*>(xs + (size_t)kt * 256 + c * 16);
                dst[0] = make_float4(a.x, a.y, b.x, b.y);
                dst[8] = make_float4(cc.x, cc.y, dd.x, dd.y);
            }
            for (int i = etid; i < FT_HG_BYTES / 16; i += FT_EPI) reinterpret_cast<uint4*>(hg)[i] = make_uint4(0u, 0u, 0u, 0u);
        } else {
            for (int i = etid; i < nkb * 64; i += FT_EPI) {
                const int kb = i >> 6, t = (i >> 3) & 7, c = i & 7;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (t < T) v = __ldg(reinterpret_cast<const uint4*>(P.x + (size_t)t * P.d + kb * 64) + c);
                *reinterpret_cast<uint4*>(xs + kb * FT_XBLOCK + t * 128 + ((c ^ t) << 4)) = v;
            }
        }
        // ---- router, step 1: the reduction over d of every token is cut into KS slices, one CTA per (token, slice).
        // A row of Wr (E floats) is covered by E/4 neighbouring threads with one 16-byte load each; a thread keeps its
        // four experts' sums over every rpp-th row of the slice; all its loads are in flight at once.
        {
            int KS = 1;
            while (KS < 16 && KS * 2 * T <= G) KS *= 2;
            const int quads = (E + 3) / 4, rpp = FT_EPI / quads;
            if ((int)blockIdx.x < T * KS) {
                const int t = blockIdx.x / KS, sl = blockIdx.x % KS;
                const int klen = (P.d + KS - 1) / KS, kbeg = sl * klen, kend = min(P.d, kbeg + klen);
                const __nv_bfloat16* __restrict__ xr = P.x + (size_t)t * P.d;
                const int qd = etid % quads, r0 = etid / quads;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r0 < rpp) {
                    if ((E & 3) == 0) {
                        for (int kb = kbeg + r0; kb < kend; kb += FT_ROUTER_BATCH * rpp) {
                            float4 w[FT_ROUTER_BATCH];
                            float xs[FT_ROUTER_BATCH];
#pragma unroll
                            for (int j = 0; j < FT_ROUTER_BATCH; ++j) {
                                const int k = kb + j * rpp;
                                const bool ok = k < kend;
                                w[j] = ok ? __ldg(reinterpret_cast<const float4*>(P.Wr + (size_t)k * E) + qd)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                                xs[j] = ok ? __bfloat162float(xr[k]) : 0.f;
                            }
#pragma unroll
                            for (int j = 0; j < FT_ROUTER_BATCH; ++j) {
                                acc.x = fmaf(xs[j], w[j].x, acc.x);
                                acc.y = fmaf(xs[j], w[j].y, acc.y);
                                acc.z = fmaf(xs[j], w[j].z, acc.z);
                                acc.w = fmaf(xs[j], w[j].w, acc.w);
                            }
                        }
                    } else {
                        const int e0 = qd * 4;
                        for (int k = kbeg + r0; k < kend; k += rpp) {
                            const float xv = __bfloat162float(xr[k]);
                            const float* w = P.Wr + (size_t)k * E + e0;
                            acc.x = fmaf(xv, __ldg(w), acc.x);
                            if (e0 + 1 < E) acc.y = fmaf(xv, __ldg(w + 1), acc.y);
                            if (e0 + 2 < E) acc.z = fmaf(xv, __ldg(w + 2), acc.z);
                            if (e0 + 3 < E) acc.w = fmaf(xv, __ldg(w + 3), acc.w);
                        }
                    }
                }
                // the threads' sums meet in shared memory (the ring is idle until the partition is known); the slice's
                // sum per expert goes to global memory, where every CTA will read it (the partial-output buffer is free
                // until the very end)
                reinterpret_cast<float4*>(smem)[etid] = acc;
                FT_SYNC();
                if (etid < E) {
                    const float* sf = reinterpret_cast<const float*>(smem);
                    float v = 0.f;
                    for (int r = 0; r < rpp; ++r) v += sf[(r * quads + (etid >> 2)) * 4 + (etid & 3)];
                    P.partial[((size_t)t * KS + sl) * kMaxExperts + etid] = v;
                }
            }
            if (etid == 0) TRACE(1);
            FT_SYNC();
            if (etid == 0) {
                grid_arrive(P.sync, 1);
                if (!grid_wait(P.sync, 1, G, &sh.abort_flag)) sh.abort_flag = 1;
                TRACE(13);
            }
            FT_SYNC();
            // ---- router, step 2, in EVERY CTA: the slices' sums of every token are fetched in one go into shared memory
            // and added per (token, expert) in ascending slice order: the same arithmetic everywhere, hence the same
            // scores, selection and partition -- nothing more to agree on
            float* stage = reinterpret_cast<float*>(smem);
            for (int i = etid; i < T * KS * E; i += FT_EPI) {
                const int e = i % E, ts = i / E;
                stage[ts * kMaxExperts + e] = __ldcg(P.partial + (size_t)ts * kMaxExperts + e);
            }
            FT_SYNC();
            for (int item = etid; item < T * E; item += FT_EPI) {
                const int t = item / E, e = item % E;
                float v = P.br ? P.br[e] : 0.f;
                for (int sl = 0; sl < KS; ++sl) v += stage[(t * KS + sl) * kMaxExperts + e];
                sh.score_s[t][e] = v;
            }
            FT_SYNC();
            // softmax and selection, one warp per token; CTA t writes token t's results out
            const int w = warp - 2;
            if (w < T) {
                const float l_lo = lane < E ? sh.score_s[w][lane] : 0.f;
                const float l_hi = lane + 32 < E ? sh.score_s[w][lane + 32] : 0.f;
                float s_lo, s_hi;
                softmax_warp(l_lo, l_hi, E, lane, s_lo, s_hi);
                const uint64_t m = select_warp(s_lo, s_hi, P.sel, lane);
                if (lane < E) sh.score_s[w][lane] = s_lo;
                if (lane + 32 < E) sh.score_s[w][lane + 32] = s_hi;
                if (lane == 0) sh.mask_s[w] = m;
                if ((int)blockIdx.x == w % G) {
                    if (lane < E) P.scores[(size_t)w * E + lane] = s_lo;
                    if (lane + 32 < E) P.scores[(size_t)w * E + lane + 32] = s_hi;
                    if (lane == 0) {
                        P.mask[w] = m;
                        if (P.k_t) P.k_t[w] = __popcll(m);
                    }
                }
            }
            ptx::fence_proxy_async();       // the scratch was read through the generic proxy; TMA writes the ring next
            FT_SYNC();
            if (etid == 0) {
                uint64_t any = 0;
                for (int t = 0; t < T; ++t) any |= sh.mask_s[t];
                int n = 0;
                for (int e = 0; e < E; ++e)
                    if ((any >> e) & 1ull) sh.active[n++] = e;
                sh.n_act = n;
                const long long U = (long long)n * upe;
                sh.u0 = (int)(U * blockIdx.x / G);
                sh.u1 = (int)(U * (blockIdx.x + 1) / G);
                int nt = 0;
                for (int u = sh.u0; u < sh.u1 && nt < FT_MAXTILES;) {
                    const int iu = u % upe, len = min(8, min(sh.u1 - u, upe - iu));
                    sh.tile_e[nt] = sh.active[u / upe];
                    sh.tile_iu0[nt] = iu;
                    sh.tile_len[nt] = len;
                    sh.tile_ul0[nt] = u - sh.u0;
                    ++nt;
                    u += len;
                }
                sh.ntiles = nt;
                sh.nchain = max(1, min(min(4, nkb), FT_TMEM_COLS / FT_N / max(nt, 1)));
                __threadfence_block();
                sh.geo_ready = 1;
                TRACE(2);
            }
            if (P.counts_out && blockIdx.x == 0 && etid < E) {
                int n = 0;
                for (int t = 0; t < T; ++t) n += (int)((sh.mask_s[t] >> etid) & 1ull);
                P.counts_out[etid] = n;
            }
            FT_SYNC();
        }
        const int nu = sh.u1 - sh.u0;
        const int q = warp & 3, grp = (warp - 2) >> 2;       // TMEM lanes 32 q ..; three warps share a quarter
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        float* mine = P.partial + (size_t)blockIdx.x * T * P.d;
        bool dead = sh.abort_flag != 0;
        if (nu > 0) {
            // ---- GeLU and gate: D1 -> shared memory, as the down-projection's token operand (16 rows of 32 bytes per
            // unit, the 32-byte swizzle written by hand)
            if (P.simt_up) {
                // Few tokens: the MMA would read 128 rows of weights per instruction at its fixed pace whatever the
                // number of tokens (about 128 cycles for 4 KB, less for a narrower tile), which is slower than the
                // memory delivers them.  The CUDA cores keep up: a row of 64 weights is read by 8 lanes (16 bytes
                // each), a warp takes 4 rows at a time, every lane keeps fp32 sums for its rows and every token.
                const int w = warp - 2, g = lane >> 3, c = lane & 7;
                int sl = 0;
                uint32_t sph = 0;
                for (int ti = 0; ti < sh.ntiles; ++ti) {
                    const int len = sh.tile_len[ti], rows = len * FT_UNIT, kbp = tmW1.kbp[len - 1];
                    float acc[3][4];
#pragma unroll
                    for (int i = 0; i < 3; ++i)
#pragma unroll
                        for (int t = 0; t < 4; ++t) acc[i][t] = 0.f;
                    for (int g0 = 0; g0 * kbp < nkb; ++g0) {
                        if (!dead && !ptx::mbar_wait(ptx::smem_u32(&sh.full[sl]), sph, &sh.abort_flag)) dead = true;
                        const uint8_t* slot = smem + sl * FT_SLOT;
                        for (int kbi = 0; !dead && kbi < kbp && g0 * kbp + kbi < nkb; ++kbi) {
                            const int kb = g0 * kbp + kbi;
                            float4 xlo[4], xhi[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                if (t < T) {
                                    const float4* xp = reinterpret_cast<const float4*>(xs + (size_t)(kb * T + t) * 256 + c * 16);
                                    xlo[t] = xp[0];
                                    xhi[t] = xp[8];
                                }
                            }
#pragma unroll
                            for (int i = 0; i < 3; ++i) {
                                const int r = 4 * (w + 12 * i) + g;
                                if (r < rows) {
                                    const uint4 wv = *reinterpret_cast<const uint4*>(slot + (size_t)kbi * rows * 128 + r * 128 +
                                                                                     ((c ^ (r & 7)) << 4));
                                    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&wv);
                                    const float2 w0 = __bfloat1622float2(h2[0]), w1 = __bfloat1622float2(h2[1]),
                                                 w2 = __bfloat1622float2(h2[2]), w3 = __bfloat1622float2(h2[3]);
#pragma unroll
                                    for (int t = 0; t < 4; ++t) {
                                        if (t < T) {
                                            float a = acc[i][t];
                                            a = fmaf(w0.x, xlo[t].x, a);
                                            a = fmaf(w0.y, xlo[t].y, a);
                                            a = fmaf(w1.x, xlo[t].z, a);
                                            a = fmaf(w1.y, xlo[t].w, a);
                                            a = fmaf(w2.x, xhi[t].x, a);
                                            a = fmaf(w2.y, xhi[t].y, a);
                                            a = fmaf(w3.x, xhi[t].z, a);
                                            a = fmaf(w3.y, xhi[t].w, a);
                                            acc[i][t] = a;
                                        }
                                    }
                                }
                            }
                        }
                        FT_SYNC();                                   // every warp is done with the slot
                        if (etid == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.empty[sl]));
                        if (++sl == FT_STAGES) {
                            sl = 0;
                            sph ^= 1u;
                        }
                    }
                    // the 8 lanes of a row add their sums; lane c = t writes token t's gated activation
                    const int e = sh.tile_e[ti];
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        const int r = 4 * (w + 12 * i) + g;
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            float v = acc[i][t];
                            v += __shfl_xor_sync(0xffffffffu, v, 1);
                            v += __shfl_xor_sync(0xffffffffu, v, 2);
                            v += __shfl_xor_sync(0xffffffffu, v, 4);
                            if (c == t && t < T && r < rows) {
                                const int ul = sh.tile_ul0[ti] + r / FT_UNIT, kk = r % FT_UNIT;
                                const float gate = ((sh.mask_s[t] >> e) & 1ull) ? sh.score_s[t][e] : 0.f;
                                *reinterpret_cast<__nv_bfloat16*>(hg + ul * (FT_N * 32) + t * 32 + ((kk >> 3) << 4) + (kk & 7) * 2) =
                                    __float2bfloat16_rn(gate * gelu_erf(v));          // rows 0..3: the swizzle leaves them in place
                            }
                        }
                    }
                }
                if (etid == 0) TRACE(6);
            } else {
            if (!dead && !ptx::mbar_wait(ptx::smem_u32(&sh.d1_full), 0u, &sh.abort_flag)) dead = true;
            dead = __any_sync(0xffffffffu, dead);
            ptx::tc_fence_after();
            if (etid == 0) TRACE(6);
            for (int ti = grp; !dead && ti < sh.ntiles; ti += 3) {
                float r[16];
#pragma unroll
                for (int t = 0; t < 16; ++t) r[t] = 0.f;
                for (int c = 0; c < sh.nchain; ++c) {
                    uint32_t rc[16];
                    ptx::tmem_ld16(tmem_base + (uint32_t)((ti * sh.nchain + c) * FT_N) + lane_base, rc);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int t = 0; t < 16; ++t) r[t] += __uint_as_float(rc[t]);
                }
                const int hr = q * 32 + lane, kk = hr % FT_UNIT;
                if (hr < sh.tile_len[ti] * FT_UNIT) {
                    const int ul = sh.tile_ul0[ti] + hr / FT_UNIT, e = sh.tile_e[ti];
                    uint8_t* dst = hg + ul * (FT_N * 32) + (kk & 7) * 2;
#pragma unroll
                    for (int t = 0; t < FT_N; ++t) {
                        float v = 0.f;
                        if (t < kFusedMaxT && t < T && ((sh.mask_s[t] >> e) & 1ull))
                            v = sh.score_s[t][e] * gelu_erf(r[t]);
                        *reinterpret_cast<__nv_bfloat16*>(dst + t * 32 + (((kk >> 3) ^ ((t >> 2) & 1)) << 4)) = __float2bfloat16_rn(v);
                    }
                }
            }
            }
            ptx::tc_fence_before();
            ptx::fence_proxy_async();           // the tensor core reads what these threads wrote
            FT_SYNC();
            if (etid == 0) {
                ptx::mbar_arrive(ptx::smem_u32(&sh.hg_ready));
                TRACE(7);
            }
            // ---- this CTA's partial output: D2 -> global memory
            if (!dead && !ptx::mbar_wait(ptx::smem_u32(&sh.d2_full), 0u, &sh.abort_flag)) dead = true;
            dead = __any_sync(0xffffffffu, dead);
            ptx::tc_fence_after();
            if (etid == 0) TRACE(9);
            for (int c = grp; !dead && c * 128 < P.d; c += 3) {
                uint32_t r[16];
                ptx::tmem_ld16(tmem_base + (uint32_t)(c * FT_N) + lane_base, r);
                ptx::tmem_ld_wait();
                const int col = c * 128 + q * 32 + lane;
                if (col < P.d) {
#pragma unroll
                    for (int t = 0; t < kFusedMaxT; ++t)
                        if (t < T) mine[(size_t)t * P.d + col] = __uint_as_float(r[t]);
                }
            }
            ptx::tc_fence_before();
        } else {
            for (int i = etid; i < T * P.d; i += FT_EPI) mine[i] = 0.f;     // no selected expert's unit fell to this CTA
        }
        // ---- grid barrier, then out[t,c] = the CTAs' partial outputs added in ascending CTA order
        FT_SYNC();
        if (etid == 0) {
            TRACE(10);
            grid_arrive(P.sync, 0);
            if (!grid_wait(P.sync, 0, G, &sh.abort_flag)) sh.abort_flag = 1;
            TRACE(11);
        }
        FT_SYNC();
        if (!sh.abort_flag) {
            // A CTA's share is `per` consecutive outputs.  Their sums over the CTAs are cut into nslice ranges of
            // CTAs, one thread per (output, range), so that all threads have loads in flight at once; the ranges'
            // sums meet in shared memory and are added in ascending order.
            const int n_out = T * P.d;
            const int per = (n_out + G - 1) / G;
            const int first = (int)blockIdx.x * per;
            const int cnt = max(0, min(per, n_out - first));
            for (int c0 = 0; c0 < cnt; c0 += FT_EPI) {
                const int w = min(FT_EPI, cnt - c0);
                const int nslice = max(1, min(16, FT_EPI / w));
                const int cps = (G + nslice - 1) / nslice;
                if (etid < w * nslice) {
                    const int o = etid % w, sl = etid / w;
                    const int b0 = sl * cps, b1 = min(G, b0 + cps);
                    const float* src = P.partial + (size_t)(first + c0 + o);
                    float sum = 0.f;
                    for (int bb = b0; bb < b1; bb += FT_FIX_BATCH) {
                        float v[FT_FIX_BATCH];
#pragma unroll
                        for (int j = 0; j < FT_FIX_BATCH; ++j)
                            v[j] = bb + j < b1 ? __ldcg(src + (size_t)(bb + j) * n_out) : 0.f;
#pragma unroll
                        for (int j = 0; j < FT_FIX_BATCH; ++j) sum += v[j];
                    }
                    red[sl * w + o] = sum;
                }
                FT_SYNC();
                if (etid < w) {
                    float sum = 0.f;
                    for (int k = 0; k < nslice; ++k) sum += red[k * w + etid];
                    if (P.out_f32) static_cast<float*>(P.out)[first + c0 + etid] = sum;
                    else static_cast<__nv_bfloat16*>(P.out)[first + c0 + etid] = __float2bfloat16_rn(sum);
                }
                FT_SYNC();
            }
        }
#undef FT_SYNC
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, FT_TMEM_COLS);
    }
#ifdef DSMOE_TRACE
    if (threadIdx.x == 0 && blockIdx.x < 192) {
        TRACE(12);
        for (int i = 0; i < 32; ++i) g_trace_fused[blockIdx.x][i] = sh.trace[i];
    }
#endif
    if (threadIdx.x == 0 && sh.abort_flag) {
        atomicExch(P.sync + 4, 1);
        if (P.dev_status) *P.dev_status = DSMOE_ERR_TIMEOUT;
    }
}

}  // namespace

#ifdef DSMOE_TRACE
extern "C" __attribute__((visibility("default"))) int dsmoe_trace_read_fused(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_trace_fused, sizeof(unsigned long long) * 192 * 32);
}
#endif

bool fused_decode_supported(const dsmoe_layer_desc& p) {
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    if (!umma_supported(p) || p.T < 1 || p.T > kFusedMaxT || p.T > G) return false;
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) return false;            // its K needs a pass over the batch first
    if (p.d > 4096 || p.d % 256) return false;       // d / 128 accumulators of 16 columns in TMEM; W2 copied in chunks of 256 columns
    return ((long long)p.E * (p.H / FT_UNIT) + G - 1) / G <= kFusedMaxUnits;
}

dsmoe_status launch_layer_fused_decode(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                       const void* packed, float* scores, uint64_t* mask, int32_t* k_t,
                                       int32_t* counts_out, void* out, char* ws, const WsLayout& L, int32_t* dev_status,
                                       cudaStream_t s) {
    DeviceState* st = nullptr;
    DSMOE_TRY(device_state(&st));
    if (!st->attr_fused) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(fused_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ft_smem_bytes(4096)));
        st->attr_fused = true;
    }
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    const BMapsUp* mW1;
    const BMapsDown* mW2;
    DSMOE_TRY(cached_bmaps_up(&mW1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_bmaps_down(&mW2, w2t, p.E, p.d, p.H));
    FusedParams P;
    P.T = p.T; P.d = p.d; P.H = p.H; P.E = p.E;
    P.x = static_cast<const __nv_bfloat16*>(x);
    P.Wr = Wr;
    P.br = br;
    P.sel = SelParams{p.E, p.mode, p.eps, p.eps_normalized, p.K, p.min_k, nullptr};
    P.scores = scores;
    P.mask = mask;
    P.k_t = k_t;
    P.counts_out = counts_out;
    P.partial = reinterpret_cast<float*>(ws + L.partial);
    P.out = out;
    P.out_f32 = p.out_fp32 ? 1 : 0;
    P.sync = reinterpret_cast<int*>(ws + L.sync);
    P.dev_status = dev_status;
#ifndef DSMOE_FUSED_SIMT_MAX_T
#define DSMOE_FUSED_SIMT_MAX_T 4
#endif
    P.simt_up = p.T <= (DSMOE_FUSED_SIMT_MAX_T < 4 ? DSMOE_FUSED_SIMT_MAX_T : 4) ? 1 : 0;
    DSMOE_CUDA_TRY(cudaMemsetAsync(P.sync, 0, 32, s));
    void* args[] = {const_cast<BMapsUp*>(mW1), const_cast<BMapsDown*>(mW2), &P};
    int timed = -1;
    DSMOE_TRY(timing_begin(s, &timed));
    DSMOE_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_decode_kernel), dim3(G), dim3(FT_THREADS),
                                               args, ft_smem_bytes(p.d), s));
    DSMOE_TRY(timing_end(s, timed));
    return DSMOE_OK;
}

}  // namespace dsmoe
