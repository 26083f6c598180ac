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
constexpr int FT_XBYTES = FT_N * 128;            // one 64-wide block of the tokens: 16 rows of 128 bytes
constexpr int FT_SLOT = FT_XBYTES + 128 * 128;   // ring slot: tokens' block + 128 rows of W1, or 512 32-byte rows of W2
constexpr int FT_STAGES = 8;
constexpr int FT_RING = FT_STAGES * FT_SLOT;     // 144 KB in flight per SM
constexpr int FT_DOWN_ROWS = 512;                // output columns per down-projection slot
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
    int* sync;               // 8 ints, zero at launch: grid-barrier counter [0] and an abort flag [4]
    int32_t* dev_status;
};

struct FShared {
    uint64_t full[FT_STAGES], empty[FT_STAGES];
    uint64_t d1_full, hg_ready, d2_full;
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int geo_ready;
    int n_act, u0, u1;                   // this CTA's units [u0, u1) of the n_act * H / 16 of the selected experts
    int active[kMaxExperts];             // the selected experts, ascending
    uint64_t mask_s[kFusedMaxT];
    float score_s[kFusedMaxT][kMaxExperts];
};
constexpr int FT_SHARED_BYTES = 4096;
static_assert(sizeof(FShared) <= FT_SHARED_BYTES, "FShared must fit its slot");
constexpr size_t FT_SMEM_BYTES = 1024 + (size_t)FT_RING + FT_HG_BYTES + FT_SHARED_BYTES + FT_RED_FLOATS * 4;
static_assert(FT_SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
static_assert(kFusedMaxT * FT_EPI * 16 <= FT_RING, "the router's scratch borrows the ring");

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
fused_decode_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ BMaps16 tmW1,
                    const __grid_constant__ BMapsK16 tmW2, const FusedParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t ring = base, hg_addr = base + FT_RING;
    uint8_t* hg = smem + FT_RING;
    FShared& sh = *reinterpret_cast<FShared*>(smem + FT_RING + FT_HG_BYTES);
    float* red = reinterpret_cast<float*>(smem + FT_RING + FT_HG_BYTES + FT_SHARED_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, T = P.T, E = P.E;
    const int upe = P.H / FT_UNIT;                       // units per expert
    const int nkb = P.d / 64;

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
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmX);
        ptx::prefetch_tensormap(&tmW2.m[2]);
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
            const int u0 = sh.u0, u1 = sh.u1, nu = u1 - u0;
            int s = 0;
            uint32_t ph = 0;
            bool alive = true;
            // up-projection: M tiles of up to 8 units (128 hidden units), every 64-wide block of d
            for (int mu0 = u0; alive && mu0 < u1; mu0 += 8) {
                const int mu1 = min(u1, mu0 + 8);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]), slot = ring + s * FT_SLOT;
                    ptx::mbar_expect_tx(bar, (uint32_t)(FT_XBYTES + (mu1 - mu0) * FT_UNIT * 128));
                    ptx::tma_load_2d(slot, &tmX, bar, kb * 64, 0);
                    // the tile's units, expert by expert (a run of units inside one expert is one copy)
                    int off = 0;
                    for (int u = mu0; u < mu1;) {
                        const int ei = u / upe, iu = u % upe, len = min(mu1 - u, upe - iu);
                        ptx::tma_load_3d_hint(slot + FT_XBYTES + off * (FT_UNIT * 128), &tmW1.m[len - 1], bar, 0,
                                              wrow(kb, iu * FT_UNIT, P.H), sh.active[ei], wpol);
                        off += len;
                        u += len;
                    }
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            // down-projection: unit by unit, 512 output columns per slot
            for (int j = 0; alive && j < nu; ++j) {
                const int u = u0 + j, e = sh.active[u / upe], hid = (u % upe) * FT_UNIT;
                const int kb = hid / 64, sub = hid % 64;
                for (int r = 0; r < P.d; r += FT_DOWN_ROWS) {
                    const int rows = min(FT_DOWN_ROWS, P.d - r);
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]), slot = ring + s * FT_SLOT;
                    ptx::mbar_expect_tx(bar, (uint32_t)rows * 32u);
                    for (int done = 0; done < rows;) {
                        const int rem = rows - done, lvl = rem >= 256 ? 2 : rem >= 128 ? 1 : 0;
                        ptx::tma_load_3d_hint(slot + done * 32, &tmW2.m[lvl], bar, sub, wrow(kb, r + done, P.d), e, wpol);
                        done += 64 << lvl;
                    }
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!alive) {
                const uint64_t t0 = ptx::globaltimer_ns();   // copies already issued still land in this CTA's smem
                while (ptx::globaltimer_ns() - t0 < 200000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && wait_geo(sh)) {
            const int u0 = sh.u0, u1 = sh.u1, nu = u1 - u0;
            const uint32_t idesc = ptx::make_idesc_bf16(128, FT_N);
            int s = 0;
            uint32_t ph = 0;
            bool alive = nu > 0;
            // D1[m][k, t] = sum over d of W1 rows (M) x tokens (N); tile m sits at TMEM columns 16 m ..
            int m = 0;
            for (int mu0 = u0; alive && mu0 < u1; mu0 += 8, ++m) {
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t slot = ring + s * FT_SLOT;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        ptx::umma_bf16(tmem_base + (uint32_t)(m * FT_N), ptx::make_desc_k_sw128(slot + FT_XBYTES + k * 32),
                                       ptx::make_desc_k_sw128(slot + k * 32), idesc, (uint32_t)((kb | k) != 0));
                    ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (alive) {
                ptx::umma_commit(ptx::smem_u32(&sh.d1_full));
                // the gated activations in shared memory (and D1 read out of TMEM: D2 takes its place)
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.hg_ready), 0u, &sh.abort_flag)) alive = false;
                ptx::tc_fence_after();
            }
            // D2[c][col, t] += W2 rows of unit j (M = 128 output columns of chunk c, K = 16) x hg of unit j (N)
            for (int j = 0; alive && j < nu; ++j) {
                for (int r = 0; r < P.d; r += FT_DOWN_ROWS) {
                    const int rows = min(FT_DOWN_ROWS, P.d - r);
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t slot = ring + s * FT_SLOT;
                    for (int c = 0; c * 128 < rows; ++c)
                        ptx::umma_bf16(tmem_base + (uint32_t)((r / 128 + c) * FT_N), make_desc_k_sw32(slot + c * 4096),
                                       make_desc_k_sw32(hg_addr + j * (FT_N * 32)), idesc, (uint32_t)(j != 0));
                    ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                    if (++s == FT_STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (alive) ptx::umma_commit(ptx::smem_u32(&sh.d2_full));
        }
    } else {
        // ------------------------------------------------------------ router, epilogues, final sum (12 warps)
        const int etid = (int)threadIdx.x - 64;
#define FT_SYNC() asm volatile("bar.sync 1, %0;" ::"n"(FT_EPI) : "memory")
        // ---- router: logits of every token.  A row of Wr (E floats) is covered by E/4 neighbouring threads with one
        // 16-byte load each; a thread keeps its four experts' sums over every rpp-th row, for every token.
        {
            const int quads = (E + 3) / 4, rpp = FT_EPI / quads;
            const int qd = etid % quads, r0 = etid / quads;
            float4 acc[kFusedMaxT];
#pragma unroll
            for (int t = 0; t < kFusedMaxT; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r0 < rpp) {
                if ((E & 3) == 0) {
                    for (int kb = r0; kb < P.d; kb += FT_ROUTER_BATCH * rpp) {
                        float4 w[FT_ROUTER_BATCH];
#pragma unroll
                        for (int j = 0; j < FT_ROUTER_BATCH; ++j) {
                            const int k = kb + j * rpp;
                            w[j] = k < P.d ? __ldg(reinterpret_cast<const float4*>(P.Wr + (size_t)k * E) + qd)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int j = 0; j < FT_ROUTER_BATCH; ++j) {
                            const int k = kb + j * rpp;
#pragma unroll
                            for (int t = 0; t < kFusedMaxT; ++t) {
                                if (t < T && k < P.d) {
                                    const float xv = __bfloat162float(P.x[(size_t)t * P.d + k]);
                                    acc[t].x = fmaf(xv, w[j].x, acc[t].x);
                                    acc[t].y = fmaf(xv, w[j].y, acc[t].y);
                                    acc[t].z = fmaf(xv, w[j].z, acc[t].z);
                                    acc[t].w = fmaf(xv, w[j].w, acc[t].w);
                                }
                            }
                        }
                    }
                } else {
                    const int e0 = qd * 4;
                    for (int k = r0; k < P.d; k += rpp) {
                        const float* w = P.Wr + (size_t)k * E + e0;
                        const float w0 = __ldg(w), w1 = e0 + 1 < E ? __ldg(w + 1) : 0.f, w2 = e0 + 2 < E ? __ldg(w + 2) : 0.f,
                                    w3 = e0 + 3 < E ? __ldg(w + 3) : 0.f;
#pragma unroll
                        for (int t = 0; t < kFusedMaxT; ++t) {
                            if (t < T) {
                                const float xv = __bfloat162float(P.x[(size_t)t * P.d + k]);
                                acc[t].x = fmaf(xv, w0, acc[t].x);
                                acc[t].y = fmaf(xv, w1, acc[t].y);
                                acc[t].z = fmaf(xv, w2, acc[t].z);
                                acc[t].w = fmaf(xv, w3, acc[t].w);
                            }
                        }
                    }
                }
            }
            // the threads' sums meet in shared memory (the ring is idle until the partition is known) and are added
            // per (token, expert) in a fixed order
            float4* scratch = reinterpret_cast<float4*>(smem);
#pragma unroll
            for (int t = 0; t < kFusedMaxT; ++t)
                if (t < T) scratch[t * FT_EPI + etid] = acc[t];
            FT_SYNC();
            const float* sf = reinterpret_cast<const float*>(smem);
            for (int item = etid; item < T * E; item += FT_EPI) {
                const int t = item / E, e = item % E;
                float v = P.br ? P.br[e] : 0.f;
                for (int r = 0; r < rpp; ++r) v += sf[((size_t)t * FT_EPI + r * quads + (e >> 2)) * 4 + (e & 3)];
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
                __threadfence_block();
                sh.geo_ready = 1;
            }
            if (P.counts_out && blockIdx.x == 0 && etid < E) {
                int n = 0;
                for (int t = 0; t < T; ++t) n += (int)((sh.mask_s[t] >> etid) & 1ull);
                P.counts_out[etid] = n;
            }
            FT_SYNC();
        }
        const int u0 = sh.u0, u1 = sh.u1, nu = u1 - u0;
        const int q = warp & 3, grp = (warp - 2) >> 2;       // TMEM lanes 32 q ..; three warps share a quarter
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        float* mine = P.partial + (size_t)blockIdx.x * T * P.d;
        bool dead = sh.abort_flag != 0;
        if (nu > 0) {
            // ---- GeLU and gate: D1 -> shared memory, as the down-projection's token operand (16 rows of 32 bytes per
            // unit, the 32-byte swizzle written by hand)
            if (!dead && !ptx::mbar_wait(ptx::smem_u32(&sh.d1_full), 0u, &sh.abort_flag)) dead = true;
            dead = __any_sync(0xffffffffu, dead);
            ptx::tc_fence_after();
            for (int m = grp; !dead && m * 8 < nu; m += 3) {
                uint32_t r[16];
                ptx::tmem_ld16(tmem_base + (uint32_t)(m * FT_N) + lane_base, r);
                ptx::tmem_ld_wait();
                const int hr = q * 32 + lane, ul = m * 8 + hr / FT_UNIT, kk = hr % FT_UNIT;
                if (ul < nu) {
                    const int e = sh.active[(u0 + ul) / upe];
                    uint8_t* dst = hg + ul * (FT_N * 32) + (kk & 7) * 2;
#pragma unroll
                    for (int t = 0; t < FT_N; ++t) {
                        float v = 0.f;
                        if (t < kFusedMaxT && t < T && ((sh.mask_s[t] >> e) & 1ull))
                            v = sh.score_s[t][e] * gelu_erf(__uint_as_float(r[t]));
                        *reinterpret_cast<__nv_bfloat16*>(dst + t * 32 + (((kk >> 3) ^ ((t >> 2) & 1)) << 4)) = __float2bfloat16_rn(v);
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::fence_proxy_async();           // the tensor core reads what these threads wrote
            FT_SYNC();
            if (etid == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.hg_ready));
            // ---- this CTA's partial output: D2 -> global memory
            if (!dead && !ptx::mbar_wait(ptx::smem_u32(&sh.d2_full), 0u, &sh.abort_flag)) dead = true;
            dead = __any_sync(0xffffffffu, dead);
            ptx::tc_fence_after();
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
            grid_arrive(P.sync, 0);
            if (!grid_wait(P.sync, 0, G, &sh.abort_flag)) sh.abort_flag = 1;
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
    if (threadIdx.x == 0 && sh.abort_flag) {
        atomicExch(P.sync + 4, 1);
        if (P.dev_status) *P.dev_status = DSMOE_ERR_TIMEOUT;
    }
}

}  // namespace

bool fused_decode_supported(const dsmoe_layer_desc& p) {
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    if (!umma_supported(p) || p.T < 1 || p.T > kFusedMaxT || p.T > G) return false;
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) return false;            // its K needs a pass over the batch first
    if (p.d > 4096) return false;                                       // d / 128 accumulators of 16 columns in TMEM
    return ((long long)p.E * (p.H / FT_UNIT) + G - 1) / G <= kFusedMaxUnits;
}

dsmoe_status launch_layer_fused_decode(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                       const void* packed, float* scores, uint64_t* mask, int32_t* k_t,
                                       int32_t* counts_out, void* out, char* ws, const WsLayout& L, int32_t* dev_status,
                                       cudaStream_t s) {
    DeviceState* st = nullptr;
    DSMOE_TRY(device_state(&st));
    if (!st->attr_fused) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(fused_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FT_SMEM_BYTES));
        st->attr_fused = true;
    }
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    const CUtensorMap* mX;
    const BMaps16* mW1;
    const BMapsK16* mW2;
    DSMOE_TRY(cached_map_2d(&mX, x, p.T, p.d, FT_N));          // rows beyond T read as zeros
    DSMOE_TRY(cached_bmaps16(&mW1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_bmaps_k16(&mW2, w2t, p.E, p.d, p.H));
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
    DSMOE_CUDA_TRY(cudaMemsetAsync(P.sync, 0, 32, s));
    void* args[] = {const_cast<CUtensorMap*>(mX), const_cast<BMaps16*>(mW1), const_cast<BMapsK16*>(mW2), &P};
    int timed = -1;
    DSMOE_TRY(timing_begin(s, &timed));
    DSMOE_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_decode_kernel), dim3(G), dim3(FT_THREADS),
                                               args, FT_SMEM_BYTES, s));
    DSMOE_TRY(timing_end(s, timed));
    return DSMOE_OK;
}

}  // namespace dsmoe
