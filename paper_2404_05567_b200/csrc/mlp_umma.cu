// Expert MLPs (Eq. 1's e(X) = GeLU(X.W1).W2) on the 5th-generation tensor cores: persistent,
// warp-specialised kernels whose operands arrive by TMA into 128-byte-swizzled shared memory, whose
// products are issued by one thread with tcgen05.mma into TMEM accumulators, and whose epilogue
// (GeLU, router gate, rounding) reads TMEM back with tcgen05.ld while the next tile's mainloop runs
// on the other half of TMEM.
//
//   warp 0      TMA producer         (one lane)
//   warp 1      MMA issuer           (one lane); owns the TMEM allocation
//   warps 2..5  epilogue             (warp w reads TMEM lanes 32*(w%4) .. +31)
//
// umma_gemm_kernel, three tilings:
//   GROUPED     rows sorted by expert (sparse inference): tile = (expert, 128 rows, <=256 columns)
//   DENSE_UP    every expert on every token (dense forward): h[t, e*H + j] = S[t,e] * GeLU(x[t].W1[e][:,j])
//   DENSE_DOWN  out[t,:] = sum over (e,j) of that h times W2[e][j,:] -- the router-weighted sum of
//               Eq. 1 folded into the reduction dimension, so no grouping and no aggregation pass
// small_layer_kernel: the whole layer for a handful of tokens (decode) in one cooperative launch.
#include <algorithm>
#include <climits>
#include <cstdlib>

#include "common.cuh"
#include "router_device.cuh"
#include "tensor_maps.cuh"
#include "umma.cuh"

namespace dsmoe {

namespace {

constexpr int BM = 128, BK = 64, BN = 256, STAGES = 4, MAX_STAGES = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int B_STAGE_BYTES = BN * BK * 2;
constexpr int NUM_THREADS = 192;
constexpr int GATHER_WARPS = 8;
constexpr int GATHER_THREADS = NUM_THREADS + 32 * GATHER_WARPS;   // umma_gemm_kernel with more warps that gather the rows of A
constexpr int SMALL_THREADS = 448;    // small_layer_kernel: 2 + 4 warps as above, plus 8 warps that share the epilogue arithmetic
constexpr int kEpiThreads = SMALL_THREADS - 64;
constexpr int TMEM_COLS = 512;
constexpr int RING_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);   // operand ring: 4 x 48 KB, or more, smaller slots
#ifndef DSMOE_SMALL_INFLIGHT
#define DSMOE_SMALL_INFLIGHT (144 * 1024)
#endif
constexpr int SMALL_RING_BYTES = DSMOE_SMALL_INFLIGHT;                 // small_layer_kernel's ring
constexpr int SHARED_BYTES = 6144 + 256;                                     // barriers and small tables (struct Shared)
#ifndef DSMOE_SMALL_STG_COLS
#define DSMOE_SMALL_STG_COLS 64
#endif
constexpr int STG_BYTES = BM * (DSMOE_SMALL_STG_COLS + 4) * 4;         // epilogue staging tile: T rows x (64..256 + 4) floats
// small_layer_kernel asks only for the ring bytes it keeps in flight: what it leaves stays with the SM's L1, which
// serves the kernel's many small loads (its parameters' copy, the router's operands)
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)SMALL_RING_BYTES + SHARED_BYTES + STG_BYTES;
constexpr size_t SMEM_GEMM_BYTES = 1024 + (size_t)RING_BYTES + SHARED_BYTES;   // umma_gemm_kernel needs no staging tile ...
// ... except with the aggregation in its epilogue: 12 epilogue warps, each with a 32 x 16 fp32 transposition tile
constexpr int CMB_WARPS = 12, CMB_COLS = 16, CMB_LD = CMB_COLS + 1;
constexpr size_t SMEM_GEMM_CMB_BYTES = SMEM_GEMM_BYTES + (size_t)CMB_WARPS * 32 * CMB_LD * 4;
static_assert(SMEM_GEMM_CMB_BYTES <= 227 * 1024, "shared memory of one CTA");

// umma_gemm_kernel comes in two forms.  Alone, a CTA computes 128 x 256 tiles from a ring of 4 slots of 16 + 32 KB.
// As a pair (a cluster of two CTAs, tcgen05 .cta_group::2), the two compute a 256 x 256 tile: each holds its own 128
// rows of A and half of the B tile's rows, the even CTA issues MMAs that read both CTAs' shared memory and write
// 128 accumulator rows into each CTA's tensor memory.  A slot is then 16 + 16 KB, so the ring holds 6 of them, and
// a CTA brings 32 KB from L2 per 64-wide reduction block instead of 48 KB.
#ifndef DSMOE_PAIR_GW
#define DSMOE_PAIR_GW 6
#endif
template <bool PAIR>
struct Geo {
    static constexpr int ST = PAIR ? 6 : STAGES;                             // ring slots
    static constexpr int B_BYTES = PAIR ? B_STAGE_BYTES / 2 : B_STAGE_BYTES; // this CTA's part of a B tile
    static constexpr int GW = PAIR ? DSMOE_PAIR_GW : GATHER_WARPS;           // warps that gather rows of A
    static constexpr int MT = PAIR ? 2 * BM : BM;                            // rows of a tile
    static_assert(ST * (A_STAGE_BYTES + B_BYTES) == RING_BYTES, "both forms fill the same ring");
    static_assert(GW % ST == 0 && ST <= MAX_STAGES, "whole warps per slot");
};

enum { GEMM_GROUPED = 0, GEMM_DENSE_UP = 1, GEMM_DENSE_DOWN = 2 };
enum { EPI_GELU = 0, EPI_STORE = 1, EPI_COMBINE = 2, EPI_BWD = 3 };
constexpr int kUpUnit = 16;          // small-T up-projection: weight rows per work unit
constexpr int kUpTileUnits = 16;     // ... and units per tile (256 rows)
constexpr int kRouterBatch = 12;     // rows of Wr a router thread loads at once
constexpr int kFixBatch = 24;        // partial tiles a fix-up thread loads at once
// small-T kernel: bytes of loads a CTA keeps in flight (<= RING_BYTES).  Four 36 KB slots per SM already cover the
// bandwidth-delay product; a deeper ring only lengthens the queues that the router's loads, the grid barriers and
// instruction fetches wait in.
constexpr int kSmallInflightBytes = SMALL_RING_BYTES;
static_assert(kSmallInflightBytes <= RING_BYTES, "in-flight bytes are ring bytes");
#ifndef DSMOE_SMALL_L2_PREFETCH
#define DSMOE_SMALL_L2_PREFETCH (384 * 1024)
#endif
constexpr int kSmallL2PrefetchBytes = DSMOE_SMALL_L2_PREFETCH;   // small-T kernel: W2 bytes a CTA asks into L2 before the middle barrier
constexpr int kSpecMinT = 8;         // tokens from which the small-T kernel streams ahead of its router

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
    // grouped, optional: row r of A is row gather[r] of the [gather_rows, k_per_expert] bf16 tensor gather_src; four
    // extra warps then fetch the A tiles themselves (the kernel is launched with GATHER_THREADS) and tmA is unused
    const int32_t* gather;
    const void* gather_src;
    int gather_rows;
    // grouped down-projection with the aggregation of Eq. 1 in its epilogue (epi == EPI_COMBINE): row r belongs to
    // token row_token[r] and carries the router gate row_gate[r]; the epilogue adds gate * (h.W2[e]) to the token's
    // fp32 running sum `acc` [tokens, n_per_expert] in ascending expert order (tile_done orders the experts), and the
    // token's last expert writes the rounded result to `out`.  With out_f32 the sum runs in `out` itself.
    const int32_t* row_token;
    const float* row_gate;
    const uint64_t* sel_mask;
    float* acc;
    int* tile_done;          // [E][column ranges], zero at launch: epilogue warps that have finished a tile
    int tokens;
    // B given in its natural layout [E][n][k] (k contiguous) instead of the packed block-major one
    int b_plain;
    // backward of the dense forward (epi == EPI_BWD, tiles as in GEMM_DENSE_UP): the accumulator holds
    // G = dO.W2[e]^T for (token, hidden unit); the epilogue writes out = gate * G (the gradient at the hidden
    // activation, Eq. 3's S_j dO passed through W2[e]) and the row's partial <act, G> over the tile's columns to
    // dot_part[(token * E + e) * column_tiles + column_tile] (Eq. 3's <e_j(X), dO>, see launch_dense_backward)
    const __nv_bfloat16* act;   // [rows, E * n_per_expert] hidden activations GeLU(x.W1[e])
    float* dot_part;
    // GEMM_DENSE_UP: "expert" e reads A's columns from e * a_expert_stride on (0: every expert reads the same columns;
    // the router's logits use it to cut their reduction into pieces with an output block each)
    int a_expert_stride;
    // GEMM_GROUPED, EPI_STORE with out_f32, single CTAs: the reduction is cut into k_splits equal runs of 64-wide blocks
    // (0 or 1: not cut); split s of a tile stores its partial sums to rows split_rows * s + r of `out`
    int k_splits, split_rows;
};

struct Tile {
    int row0, rows_valid, e, n0, bn, nk, out_col0;   // rows_valid <= 0: this CTA's half of a pair's tile lies past the rows
    int row_safe;                                    // a row that exists (stands in for rows past the end)
    int k0, out_row0;                                // first 64-wide block of the reduction; row of `out` that row0 goes to
};

// small_layer_kernel: the selected experts and the work partition and ring geometry that follow from them
struct SmallGeo {
    int n_act;                           // experts selected by at least one token
    int up_rows, bn_down;                // widest up-projection tile; column-range width of the down-projection
    int a_bytes, slot_bytes, n_stages;   // ring: token block + weight tile per slot
    int active[kMaxExperts];             // their indices, ascending
};

struct Shared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tfull[2], tempty[2];
    uint64_t drain;                      // small_layer_kernel: "every MMA on speculative tiles has completed"
    uint32_t tmem_base;
    volatile int abort_flag;
    int bad_offsets;
    int tile_prefix[kMaxExperts + 1];
    int seg0[kMaxExperts], seg1[kMaxExperts];
    unsigned long long active_mask;
    // small_layer_kernel: geo[0] assumes every expert selected (streaming starts under it while the router still
    // runs), geo[1] is what the router found.  geo_state: 0 router pending; 1 the up-projection started under geo[0] stands (geo[1]
    // equals it, or misses only a few experts and has the same ring: their tiles are computed for nothing and gated
    // to zero); 2 it is started over under geo[1].
    SmallGeo geo[2];
    volatile int up_geo;                   // which of the two the up-projection follows (the down-projection: always geo[1])
    volatile int geo_state;
    volatile int spec_issued, spec_stop;   // producer -> MMA issuer: ring slots filled under geo[0]; no more will be
    volatile int up_arrived;               // epilogue -> producer: this CTA has arrived at the barrier between the projections
    volatile int mma_drained;              // MMA issuer -> producer: those slots are consumed, the ring is idle
    union {
        int rowtok[(DSMOE_PAIR_GW > 8 ? DSMOE_PAIR_GW / 2 : 6) * BM];                // umma_gemm_kernel, gathered A: the source row of each tile row, per gathering warp
        struct {                           // small_layer_kernel: router gates and every token's selection word
            float gate_s[BM], gate2_s[BM];
            uint64_t mask_s[BM];
        };
    };
#ifdef DSMOE_TRACE
    unsigned long long trace[32];
#endif
};
static_assert(sizeof(Shared) <= SHARED_BYTES, "Shared must fit its slot");

#ifdef DSMOE_TRACE
// Diagnostic build only (-DDSMOE_TRACE): per-CTA time stamps (globaltimer ns) of small_layer_kernel's milestones.
__device__ unsigned long long g_trace[192][32];
#define TRACE(i) sh.trace[i] = ptx::globaltimer_ns()
// ... and of umma_gemm_kernel: clock cycles its roles spent waiting, per CTA, for the last launch of each kind
// (0 router logits, 1 up-projection, 2 down-projection or backward): [0] MMA issuer in all, [1] of these waiting for
// operands, [2] for a free accumulator; [3] producer in all, [4] of these waiting for a free slot; [5] first epilogue
// warp in all, [6] of these waiting for an accumulator; [7] tiles
__device__ long long g_gemm_trace[3][192][8];
#define GTRACE_T0(v) const long long v = clock64()
#define GTRACE_ADD(slot, v) gtr[slot] += clock64() - (v)
#else
#define TRACE(i)
#define GTRACE_T0(v)
#define GTRACE_ADD(slot, v)
#endif

// GeLU(v) = v Phi(v) with the exact Phi (the erf form, not the tanh form).  Phi comes from Abramowitz & Stegun's
// rational approximation 7.1.28, erfc(z) = (1 + a1 z + ... + a6 z^6)^-16 with |error| <= 3e-7 for z >= 0 -- three
// orders below the bf16 rounding of the result: Phi(v) = erfc(|v| / sqrt 2) / 2 for v < 0 and 1 minus that for
// v >= 0, so the negative tail has no cancellation.  Six FMAs, one reciprocal, four squarings: about half the
// instructions of erff, which matters because the GeLU epilogue of a tile costs the CUDA cores nearly as many issue
// slots as its mainloop costs the tensor core.
__device__ __forceinline__ float gelu_erf(float v) {
    const float z = fabsf(v) * 0.70710678118654752440f;
    float p = fmaf(z, 0.0000430638f, 0.0002765672f);
    p = fmaf(z, p, 0.0001520143f);
    p = fmaf(z, p, 0.0092705272f);
    p = fmaf(z, p, 0.0422820123f);
    p = fmaf(z, p, 0.0705230784f);
    p = fmaf(z, p, 1.f);
    float q;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(q) : "f"(p));   // p >= 1: one unit in the last place is plenty
    q *= q;
    q *= q;
    q *= q;
    q *= q;
    const float tail = 0.5f * q;                    // Phi(-|v|)
    return v * (v < 0.f ? tail : 1.f - tail);
}

// The packed weights are block-major along the reduction: [E][k / 64][n][64], so the tile (64 k, rows n0..) of
// reduction block kb is the `rows` consecutive 128-byte rows starting at wrow(kb, n0, N) of a [E][(K/64)*N][64]
// tensor: one contiguous piece of memory.
__device__ __forceinline__ int wrow(int kb, int n0, int N) { return kb * N + n0; }

// Weight rows [row0, row0 + rows) of expert e (see wrow): power-of-two boxes, largest first.
template <bool PAIR = false>
__device__ __forceinline__ void load_weight_rows(const BMaps* maps, uint32_t dst, uint32_t bar, int row0, int rows,
                                                 int e, int x0 = 0) {
    int done = 0;
#pragma unroll
    for (int lvl = 4; lvl >= 0; --lvl) {
        if ((rows - done) >= (16 << lvl)) {
            if (PAIR) ptx::tma_load_3d_pair(dst + done * (BK * 2), &maps->m[lvl], bar, x0, row0 + done, e);
            else ptx::tma_load_3d(dst + done * (BK * 2), &maps->m[lvl], bar, x0, row0 + done, e);
            done += 16 << lvl;
        }
    }
}

constexpr long long kUpBandBytes = 24ll << 20;     // dense up-projection: rows of A that one band of row tiles may hold

template <bool PAIR>
__device__ __forceinline__ int total_tiles(const GemmParams& P, const Shared& sh) {
    constexpr int MT = Geo<PAIR>::MT;
    const int ntn = (P.n_per_expert + BN - 1) / BN;
    if (P.mode == GEMM_GROUPED) return sh.tile_prefix[P.E] * max(P.k_splits, 1);
    const int mt = (P.rows + MT - 1) / MT;
    return P.mode == GEMM_DENSE_UP ? mt * ntn * P.E : mt * ntn;
}

// Tile `id` as CTA `half` (0, or 1 for the odd CTA of a pair) sees it: its own 128 rows, the whole column range.
template <bool PAIR>
__device__ __forceinline__ Tile decode_tile(const GemmParams& P, const Shared& sh, int id, int half) {
    constexpr int MT = Geo<PAIR>::MT;
    Tile t;
    const int kbpe = P.k_per_expert / BK;
    t.k0 = 0;
    if (P.mode == GEMM_GROUPED) {
        const int splits = max(P.k_splits, 1), split = id % splits;
        id /= splits;
        int e = 0;
        while (e + 1 < P.E && id >= sh.tile_prefix[e + 1]) ++e;
        const int local = id - sh.tile_prefix[e];
        const int cnt = sh.seg1[e] - sh.seg0[e];
        const int mtiles = (cnt + MT - 1) / MT;
        const int nt = local / mtiles, mt = local % mtiles;
        t.e = e;
        t.row0 = sh.seg0[e] + mt * MT + half * BM;
        t.rows_valid = min(BM, sh.seg1[e] - t.row0);
        t.row_safe = sh.seg0[e];
        t.n0 = nt * BN;
        t.nk = kbpe / splits;
        t.k0 = split * t.nk;
        t.out_col0 = t.n0;
        t.out_row0 = t.row0 + split * P.split_rows;
    } else {
        const int mtiles = (P.rows + MT - 1) / MT;
        const int ntn = (P.n_per_expert + BN - 1) / BN;
        // Dense down: column
        // ranges fastest, so they share a few row tiles of A (every expert's hidden activations, far larger than L2,
        // which would otherwise stream from DRAM once per column range) and all of the weights.
        const bool n_first = P.mode == GEMM_DENSE_DOWN;
        int mt, rest;
        if (n_first) {
            mt = id / ntn;
            rest = id % ntn;
        } else {
            // Bands of row tiles whose rows of A (x) stay in L2 while every expert's weight tiles pass by once per band;
            // inside a band row tiles go fastest, so the CTAs running at one time share a weight tile.  (With one band
            // over all rows, x -- larger than what L2 keeps beside the hg stream -- came back from DRAM some 30 times:
            // C4 up-projection 1.87 -> 1.73 ms, the gradients' two launches 3.90 -> 3.50 ms.)
            const int band_m = max(1, min(mtiles, (int)(kUpBandBytes / ((long long)MT * P.k_per_expert * 2))));
            const int per_band = band_m * ntn * P.E;
            const int band = id / per_band, rem = id % per_band;
            const int bm = min(band_m, mtiles - band * band_m);
            mt = band * band_m + rem % bm;
            rest = rem / bm;
        }
        t.row0 = mt * MT + half * BM;
        t.out_row0 = t.row0;
        t.rows_valid = min(BM, P.rows - t.row0);
        t.row_safe = 0;
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

// Bounded wait until the int at `flag` (written by other CTAs with a release fence before it) is at least
// `target`.  false = gave up (limit reached, or another thread of the CTA already had).
__device__ __forceinline__ bool flag_wait_ge(const int* flag, int target, volatile int* abort_flag) {
    uint64_t t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v >= target) return true;
        if ((spin & 0x3f) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > ptx::kWaitLimitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

// A barrier of this CTA that (in a pair) the other CTA or its tensor core also signals
template <bool PAIR>
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return PAIR ? ptx::mbar_wait_cluster(bar, parity, abort_flag) : ptx::mbar_wait(bar, parity, abort_flag);
}

template <bool PAIR>
__global__ void __launch_bounds__((PAIR && NUM_THREADS + 32 * DSMOE_PAIR_GW > GATHER_THREADS) ? NUM_THREADS + 32 * DSMOE_PAIR_GW : GATHER_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ BMaps tmB, const GemmParams P) {
    constexpr int ST = Geo<PAIR>::ST, B_BYTES = Geo<PAIR>::B_BYTES, GW = Geo<PAIR>::GW, MT = Geo<PAIR>::MT;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;             // 128-byte swizzle wants 1024-byte aligned tiles
    const uint32_t smA = base, smB = base + ST * A_STAGE_BYTES;
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw + (base - raw) + RING_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // pair: `half` is this CTA's place in it (0 issues the MMAs and owns the barriers both CTAs signal); the pair
    // walks the tiles pair_id, pair_id + pairs, ...
    const int half = PAIR ? (int)ptx::cluster_ctarank() : 0;
    const int first_tile = PAIR ? (int)blockIdx.x / 2 : (int)blockIdx.x;
    const int tile_step = PAIR ? (int)gridDim.x / 2 : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < ST; ++s) {
            // the producer's arrival (pair: the even CTA's) + one per gathering warp of the slot (pair: of either CTA)
            const int gather_arrivals = (PAIR ? 2 : 1) * (GW / ST);
            ptx::mbar_init(ptx::smem_u32(&sh.full[s]), P.gather ? 1 + gather_arrivals : 1);
            ptx::mbar_init(ptx::smem_u32(&sh.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_u32(&sh.tfull[a]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.tempty[a]), (P.epi == EPI_COMBINE ? CMB_WARPS : 4) * (PAIR ? 2 : 1));
        }
        sh.abort_flag = 0;
        sh.bad_offsets = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmA);
        for (int i = 2; i < 5; ++i) ptx::prefetch_tensormap(&tmB.m[i]);
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
            run += ((sh.seg1[e] - sh.seg0[e] + MT - 1) / MT) * ntn;
        }
        sh.tile_prefix[P.E] = run;
    }
    if (warp == 1) {
        if (PAIR) {
            ptx::tmem_alloc_pair(ptx::smem_u32(&sh.tmem_base), TMEM_COLS);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), TMEM_COLS);
            ptx::tmem_relinquish();
        }
    }
    ptx::tc_fence_before();
    if (PAIR) ptx::cluster_sync();      // both CTAs' barriers and tensor memory exist before either signals the other
    else __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;
    const int ntiles = total_tiles<PAIR>(P, sh);
    const int kbpe = P.k_per_expert / BK;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool alive = true;
#ifdef DSMOE_TRACE
            long long gtr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
            GTRACE_T0(t_all);
            for (int id = first_tile; id < ntiles && alive; id += tile_step) {
                const Tile t = decode_tile<PAIR>(P, sh, id, half);
                for (int i = 0; i < t.nk; ++i) {
                    GTRACE_T0(t_w);
                    if (!bar_wait<PAIR>(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    GTRACE_ADD(4, t_w);
                    // pair: the bytes of both CTAs' copies are counted at the even CTA's barrier, which its producer arms
                    const uint32_t bar = PAIR ? ptx::map_to_cta(ptx::smem_u32(&sh.full[s]), 0) : ptx::smem_u32(&sh.full[s]);
                    const uint32_t bytes = (P.gather ? 0u : (uint32_t)A_STAGE_BYTES) + (uint32_t)t.bn * BK * 2;
                    if (!PAIR) ptx::mbar_expect_tx(bar, bytes);
                    else if (half == 0) ptx::mbar_expect_tx(ptx::smem_u32(&sh.full[s]), bytes + (P.gather ? 0u : (uint32_t)A_STAGE_BYTES));
                    int a_col, b_e, b_k;
                    if (P.mode == GEMM_DENSE_DOWN) {
                        b_e = i / kbpe;
                        b_k = (i % kbpe) * BK;
                        a_col = b_e * P.k_per_expert + b_k;
                    } else {
                        b_e = t.e;
                        b_k = (t.k0 + i) * BK;
                        a_col = t.e * P.a_expert_stride + b_k;
                    }
                    if (!P.gather) {
                        if (PAIR) ptx::tma_load_2d_pair(smA + s * A_STAGE_BYTES, &tmA, bar, a_col, t.row0);
                        else ptx::tma_load_2d(smA + s * A_STAGE_BYTES, &tmA, bar, a_col, t.row0);
                    }
                    // full-width tiles take the one 256-row copy (pair: this CTA's 128 rows) directly (measurably
                    // faster than walking the box sizes); only a ragged last column tile needs the decomposition
                    const int b_x = P.b_plain ? b_k : 0;
                    const int b_rows = PAIR ? t.bn / 2 : t.bn;
                    const int b_row = (P.b_plain ? t.n0 : wrow(b_k / BK, t.n0, P.n_per_expert)) + half * b_rows;
                    if (t.bn == BN) {
                        if (PAIR) ptx::tma_load_3d_pair(smB + s * B_BYTES, &tmB.m[3], bar, b_x, b_row, b_e);
                        else ptx::tma_load_3d(smB + s * B_BYTES, &tmB.m[4], bar, b_x, b_row, b_e);
                    } else {
                        load_weight_rows<PAIR>(&tmB, smB + s * B_BYTES, bar, b_row, b_rows, b_e, b_x);
                    }
                    if (++s == ST) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
#ifdef DSMOE_TRACE
            GTRACE_ADD(3, t_all);
            if (blockIdx.x < 192) {
                long long* g = g_gemm_trace[P.epi == EPI_GELU ? 1 : (P.n_per_expert <= 192 ? 0 : 2)][blockIdx.x];
                g[3] = gtr[3];
                g[4] = gtr[4];
            }
#endif
            if (!alive) {
                // copies already issued still land in this CTA's shared memory: give them time
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 200000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && half == 0) {
            int s = 0, acc = 0;
            uint32_t ph = 0, aph = 0;
            bool alive = true;
#ifdef DSMOE_TRACE
            long long gtr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
            GTRACE_T0(t_all);
            for (int id = first_tile; id < ntiles && alive; id += tile_step) {
                const Tile t = decode_tile<PAIR>(P, sh, id, 0);
                GTRACE_T0(t_acc);
                if (!bar_wait<PAIR>(ptx::smem_u32(&sh.tempty[acc]), aph ^ 1u, &sh.abort_flag)) break;
                GTRACE_ADD(2, t_acc);
#ifdef DSMOE_TRACE
                gtr[7] += 1;
#endif
                ptx::tc_fence_after();
                const uint32_t idesc = ptx::make_idesc_bf16(MT, (uint32_t)t.bn);
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int i = 0; i < t.nk; ++i) {
                    GTRACE_T0(t_w);
                    if (!bar_wait<PAIR>(ptx::smem_u32(&sh.full[s]), ph, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    GTRACE_ADD(1, t_w);
                    ptx::tc_fence_after();
                    const uint32_t a0 = smA + s * A_STAGE_BYTES, b0 = smB + s * B_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        if (PAIR)
                            ptx::umma_bf16_pair(d_tmem, ptx::make_desc_k_sw128(a0 + k * 32), ptx::make_desc_k_sw128(b0 + k * 32),
                                                idesc, (uint32_t)((i | k) != 0));
                        else
                            ptx::umma_bf16(d_tmem, ptx::make_desc_k_sw128(a0 + k * 32), ptx::make_desc_k_sw128(b0 + k * 32),
                                           idesc, (uint32_t)((i | k) != 0));
                    }
                    // slot reusable once these MMAs have read it (pair: in both CTAs)
                    if (PAIR) {
                        ptx::umma_commit_pair(ptx::smem_u32(&sh.empty[s]));
                        ptx::umma_commit_pair(ptx::map_to_cta(ptx::smem_u32(&sh.empty[s]), 1));
                    } else {
                        ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                    }
                    if (++s == ST) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (!alive) break;
                // accumulator complete (pair: each CTA's epilogue reads its own 128 rows)
                if (PAIR) {
                    ptx::umma_commit_pair(ptx::smem_u32(&sh.tfull[acc]));
                    ptx::umma_commit_pair(ptx::map_to_cta(ptx::smem_u32(&sh.tfull[acc]), 1));
                } else {
                    ptx::umma_commit(ptx::smem_u32(&sh.tfull[acc]));
                }
                if (++acc == 2) {
                    acc = 0;
                    aph ^= 1u;
                }
            }
#ifdef DSMOE_TRACE
            GTRACE_ADD(0, t_all);
            if (blockIdx.x < 192) {
                long long* g = g_gemm_trace[P.epi == EPI_GELU ? 1 : (P.n_per_expert <= 192 ? 0 : 2)][blockIdx.x];
                g[0] = gtr[0];
                g[1] = gtr[1];
                g[2] = gtr[2];
                g[7] = gtr[7];
            }
#endif
        }
    } else if (warp >= 6 && P.gather) {
        // ------------------------------------------------------------ gather (grouped up-projection only)
        // Alone, 8 warps: warps j and j + 4 bring the two halves of the A tiles of the ring stages j, j + 4, ... of
        // this CTA's sequence; in a pair, 6 warps: warp j brings the whole A tile of the stages j, j + 6, ....  An
        // instruction covers 4 rows x 128 bytes (8 lanes x 16 bytes per row), written in the 128-byte-swizzle order
        // the MMA descriptors expect (chunk c of row r sits at chunk c ^ (r % 8)).  The warp then waits for its
        // copies, makes them visible to the tensor core's proxy and arrives at the stage's barrier; while it
        // waits, the other warps' stages are in flight.
        if (warp >= 6 + GW) goto teardown;
        constexpr int PARTS = GW / ST, ROWS = BM / PARTS;   // warps per stage, rows per warp
        const int team = (warp - 6) % ST, part = (warp - 6) / ST;
        int* rowtok = sh.rowtok + (warp - 6) * ROWS;
        const int lr = lane >> 3, lc = lane & 7;
        int n = 0;                       // stages of the sequence seen so far
        bool alive = true;
        for (int id = first_tile; id < ntiles && alive; id += tile_step) {
            const Tile t = decode_tile<PAIR>(P, sh, id, half);
            __syncwarp();
#pragma unroll
            for (int j = 0; j < ROWS / 32; ++j) {
                const int r = part * ROWS + lane + 32 * j;
                const int tok = P.gather[r < t.rows_valid ? t.row0 + r : t.row_safe];   // rows past the segment: nobody reads them
                rowtok[lane + 32 * j] = min(max(tok, 0), P.gather_rows - 1);
            }
            __syncwarp();
            // this lane's rows (4 jj + lane / 8 of the warp's share): where they start in the source, in 16-byte units
            uint32_t src_off[ROWS / 4];
#pragma unroll
            for (int jj = 0; jj < ROWS / 4; ++jj)
                src_off[jj] = (uint32_t)(((size_t)rowtok[jj * 4 + lr] * P.k_per_expert * 2) >> 4);
            for (int i = 0; i < t.nk; ++i, ++n) {
                if (n % ST != team) continue;
                const int s = n % ST;
                const uint32_t ph = (uint32_t)(n / ST) & 1u;
                if (!bar_wait<PAIR>(ptx::smem_u32(&sh.empty[s]), ph ^ 1u, &sh.abort_flag)) {
                    alive = false;
                    break;
                }
                const uint32_t dst0 = smA + s * A_STAGE_BYTES;
                const char* src0 = static_cast<const char*>(P.gather_src) + (size_t)(t.k0 + i) * (BK * 2) + lc * 16;
#pragma unroll
                for (int jj = 0; jj < ROWS / 4; ++jj) {
                    const int rl = jj * 4 + lr, r = part * ROWS + rl;
                    ptx::cp_async16(dst0 + (uint32_t)r * (BK * 2) + (uint32_t)((lc ^ (r & 7)) << 4),
                                    src0 + ((size_t)src_off[jj] << 4));
                }
                ptx::cp_async_commit();
                ptx::cp_async_wait<0>();
                ptx::fence_proxy_async();
                __syncwarp();              // every lane's rows are in place and fenced: one arrival for the warp
                if (lane == 0) {
                    if (PAIR) ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&sh.full[s]), 0));
                    else ptx::mbar_arrive(ptx::smem_u32(&sh.full[s]));
                }
            }
        }
    } else if (warp < 6 || P.epi == EPI_COMBINE) {
        // ------------------------------------------------------------ epilogue (4 warps; 12 with the aggregation)
        const int q = warp & 3;
        int acc = 0;
        uint32_t aph = 0;
        // pair: the accumulators are free again once both CTAs' epilogues have read them; the even CTA's issuer waits
        const auto release_acc = [&](int a) {
            if (PAIR) ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&sh.tempty[a]), 0));
            else ptx::mbar_arrive(ptx::smem_u32(&sh.tempty[a]));
        };
#ifdef DSMOE_TRACE
        long long gtr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
        GTRACE_T0(t_all);
        for (int id = first_tile; id < ntiles; id += tile_step) {
            const Tile t = decode_tile<PAIR>(P, sh, id, half);
            // the TMEM reads below are warp-collective: the warp leaves as one
            GTRACE_T0(t_w);
            if (__any_sync(0xffffffffu, !bar_wait<PAIR>(ptx::smem_u32(&sh.tfull[acc]), aph, &sh.abort_flag))) break;
            GTRACE_ADD(6, t_w);
            ptx::tc_fence_after();
            const int row = q * 32 + lane;
            const bool valid = row < t.rows_valid;
            const long long grow = (long long)t.row0 + row;
            float g = 1.f;
            if (P.gate && valid) g = P.gate[grow * P.E + t.e];
            if (P.epi == EPI_STORE && P.row_gate && valid) g = P.row_gate[grow];
            const uint32_t taddr = tmem_base + (uint32_t)(acc * BN) + ((uint32_t)(q * 32) << 16);
            const bool warp_has_rows = q * 32 < t.rows_valid;   // warps without a valid row skip the read-back
            if (P.epi == EPI_COMBINE) {
                // Aggregation fused into the down-projection.  A token's experts add their outputs to its running
                // sum one after the other, lowest expert first -- the order of the separate aggregation kernel, so
                // the result is the same bit for bit and run to run.  That order holds because this tile only
                // touches the sums once every tile of the previous non-empty expert that covers the same columns has
                // finished (tiles are handed out in ascending expert order to CTAs that are all resident: the
                // wait is for work that is already running or done).
                // Three warps share each quarter of the accumulator's rows (a warp reads TMEM lanes 32 (warp % 4) ..),
                // taking every third 16-column piece: 12 warps' worth of loads of the old sums are in flight.  A
                // piece goes from TMEM (lane = row) through a small shared-memory tile into a layout in which 4
                // neighbouring lanes hold one row's 64 bytes, so that the sums are read and written in full sectors.
                const int ntn = (P.n_per_expert + BN - 1) / BN, nt = t.n0 / BN;
                const int slot = warp < 6 ? 0 : 1 + (warp - 6) / 4;
                float* tp = reinterpret_cast<float*>(smem_raw + (base - raw) + RING_BYTES + SHARED_BYTES) +
                            (slot * 4 + q) * 32 * CMB_LD;
                int prev = t.e - 1;
                while (prev >= 0 && sh.seg1[prev] <= sh.seg0[prev]) --prev;
                bool ok = true;
                if (prev >= 0 && warp_has_rows) {
                    if (lane == 0) {
                        const int target = CMB_WARPS * (PAIR ? 2 : 1) * ((sh.seg1[prev] - sh.seg0[prev] + MT - 1) / MT);
                        ok = flag_wait_ge(P.tile_done + prev * ntn + nt, target, &sh.abort_flag);
                    }
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                }
                if (!ok) break;
                // this lane's own row (lane = row): token, gate, and whether the expert is the token's first / last
                int tok = 0, flags = 0;
                float g = 0.f;
                if (valid) {
                    tok = min(max(P.row_token[grow], 0), P.tokens - 1);
                    g = P.row_gate[grow];
                    const uint64_t m = P.sel_mask[tok];
                    flags = 4 | ((m & ((1ull << t.e) - 1ull)) == 0ull ? 1 : 0) | (((m >> t.e) >> 1) == 0ull ? 2 : 0);
                }
                // ... and the same for the four rows this lane serves in the transposed layout: rows rg + 8 i,
                // 16-byte piece pc of their 64 bytes
                const int rg = lane >> 2, pc = lane & 3;
                int tk[4], fl[4];
                float gt[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    tk[i] = __shfl_sync(0xffffffffu, tok, rg + 8 * i);
                    fl[i] = __shfl_sync(0xffffffffu, flags, rg + 8 * i);
                    gt[i] = __shfl_sync(0xffffffffu, g, rg + 8 * i);
                }
                const int npieces = t.bn / CMB_COLS;
                auto fetch = [&](int piece, float4 (&o)[4]) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (piece < npieces && (fl[i] & 5) == 4)      // a valid row that is not its token's first expert
                            o[i] = __ldcg(reinterpret_cast<const float4*>(
                                P.acc + (long long)tk[i] * P.n_per_expert + t.out_col0 + piece * CMB_COLS + pc * 4));
                    }
                };
                float4 cur[4], nxt[4];
                if (warp_has_rows) fetch(slot, cur);
                for (int piece = slot; warp_has_rows && piece < npieces; piece += CMB_WARPS / 4) {
                    fetch(piece + CMB_WARPS / 4, nxt);
                    uint32_t r[16];
                    ptx::tmem_ld16(taddr + (uint32_t)(piece * CMB_COLS), r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) tp[lane * CMB_LD + j] = __uint_as_float(r[j]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float* src = tp + (rg + 8 * i) * CMB_LD + pc * 4;
                        float4 v = cur[i];
                        v.x = fmaf(gt[i], src[0], v.x);
                        v.y = fmaf(gt[i], src[1], v.y);
                        v.z = fmaf(gt[i], src[2], v.z);
                        v.w = fmaf(gt[i], src[3], v.w);
                        if (!(fl[i] & 4)) continue;
                        const long long o = (long long)tk[i] * P.n_per_expert + t.out_col0 + piece * CMB_COLS + pc * 4;
                        if ((fl[i] & 2) && !P.out_f32) {
                            uint2 pk;
                            *reinterpret_cast<__nv_bfloat162*>(&pk.x) = __floats2bfloat162_rn(v.x, v.y);
                            *reinterpret_cast<__nv_bfloat162*>(&pk.y) = __floats2bfloat162_rn(v.z, v.w);
                            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(P.out) + o) = pk;
                        } else {
                            __stcg(reinterpret_cast<float4*>(P.acc + o), v);
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    release_acc(acc);
                    __threadfence();                       // the warp's sums are visible before its arrival is
                    atomicAdd(P.tile_done + t.e * ntn + nt, 1);
                }
                if (++acc == 2) {
                    acc = 0;
                    aph ^= 1u;
                }
                continue;
            }
            if (P.epi == EPI_BWD) {
                const bool active = valid && (!P.sel_mask || ((P.sel_mask[grow] >> t.e) & 1ull));   // Eq. 2's mask M
                const float gs = active ? g : 0.f;
                float dot = 0.f;
                // the activations come in and the gradients go out through two shared-memory tiles, whole rows per
                // load / store instruction (4 lanes a row's 64 bytes, eight rows at a time)
                constexpr int LDB = 80;                 // bytes per staged row
                unsigned char* ta = smem_raw + (base - raw) + RING_BYTES + SHARED_BYTES + q * 2 * 32 * LDB;
                unsigned char* tb = ta + 32 * LDB;
                const int rr = lane >> 2, cc = lane & 3;
                const __nv_bfloat16* const act = P.act;
                __nv_bfloat16* const out_h = static_cast<__nv_bfloat16*>(P.out);
                for (int c = 0; warp_has_rows && c < t.bn; c += 32) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rl = i * 8 + rr;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (q * 32 + rl < t.rows_valid)
                            v = __ldg(reinterpret_cast<const uint4*>(act + ((long long)t.row0 + q * 32 + rl) * P.ld_out + t.out_col0 + c + cc * 8));
                        *reinterpret_cast<uint4*>(ta + rl * LDB + 16 * cc) = v;
                    }
                    uint32_t r[32];
                    ptx::tmem_ld32(taddr + (uint32_t)c, r);
                    ptx::tmem_ld_wait();
                    __syncwarp();
                    uint4 av[4], pk[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) av[j] = *reinterpret_cast<const uint4*>(ta + lane * LDB + 16 * j);
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
                    const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(av);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float g0 = __uint_as_float(r[2 * j]), g1 = __uint_as_float(r[2 * j + 1]);
                        if (active) {
                            const float2 a = __bfloat1622float2(ah[j]);
                            dot = fmaf(a.x, g0, dot);
                            dot = fmaf(a.y, g1, dot);
                        }
                        hv[j] = __floats2bfloat162_rn(gs * g0, gs * g1);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(tb + lane * LDB + 16 * j) = pk[j];
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rl = i * 8 + rr;
                        if (q * 32 + rl < t.rows_valid)
                            *reinterpret_cast<uint4*>(out_h + ((long long)t.row0 + q * 32 + rl) * P.ld_out + t.out_col0 + c + cc * 8) =
                                *reinterpret_cast<const uint4*>(tb + rl * LDB + 16 * cc);
                    }
                    __syncwarp();
                }
                if (valid) {
                    const int ntn = (P.n_per_expert + BN - 1) / BN;
                    P.dot_part[(grow * P.E + t.e) * ntn + t.n0 / BN] = active ? dot : 0.f;
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) release_acc(acc);
                if (++acc == 2) {
                    acc = 0;
                    aph ^= 1u;
                }
                continue;
            }
            // EPI_GELU and EPI_STORE.  The rows go out through a shared-memory tile.
            if (P.out_f32) {
                // fp32 rows: out of TMEM a lane holds 32 columns of ONE row (128 bytes that
                // it would store as eight scattered 16-byte pieces); turned through the tile, 8 lanes store one row's 128
                // bytes together, four whole rows per instruction
                constexpr int LD = 36;                  // floats per staged row: 16-byte aligned, conflict-free in quarter warps
                float* tp = reinterpret_cast<float*>(smem_raw + (base - raw) + RING_BYTES + SHARED_BYTES) + q * 32 * LD;
                const int rr = lane >> 3, cc = lane & 7;
                float* const out_f = static_cast<float*>(P.out);
                for (int c = 0; warp_has_rows && c < t.bn; c += 32) {
                    uint32_t r[32];
                    ptx::tmem_ld32(taddr + (uint32_t)c, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4*>(tp + lane * LD + 4 * j) =
                            make_float4(g * __uint_as_float(r[4 * j]), g * __uint_as_float(r[4 * j + 1]),
                                        g * __uint_as_float(r[4 * j + 2]), g * __uint_as_float(r[4 * j + 3]));
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rl = i * 4 + rr;      // row of this warp's 32
                        if (q * 32 + rl < t.rows_valid)
                            *reinterpret_cast<float4*>(out_f + ((long long)t.out_row0 + q * 32 + rl) * P.ld_out + t.out_col0 + c + cc * 4) =
                                *reinterpret_cast<const float4*>(tp + rl * LD + cc * 4);
                    }
                    __syncwarp();
                }
            } else {
                // bf16 rows (hidden activations, bf16 outputs) the same way: a lane's 64 bytes of one row go through the
                // tile, 4 lanes store a row's 64 bytes together, eight rows per instruction
                constexpr int LDB = 80;                 // bytes per staged row
                unsigned char* tb = smem_raw + (base - raw) + RING_BYTES + SHARED_BYTES + q * 32 * LDB;
                const int rr = lane >> 2, cc = lane & 3;
                __nv_bfloat16* const out_h = static_cast<__nv_bfloat16*>(P.out);
                for (int c = 0; warp_has_rows && c < t.bn; c += 32) {
                    uint32_t r[32];
                    ptx::tmem_ld32(taddr + (uint32_t)c, r);
                    ptx::tmem_ld_wait();
                    uint4 pk[4];
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(pk);
                    if (P.epi == EPI_GELU) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            hv[j] = __floats2bfloat162_rn(g * gelu_erf(__uint_as_float(r[2 * j])),
                                                          g * gelu_erf(__uint_as_float(r[2 * j + 1])));
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            hv[j] = __floats2bfloat162_rn(g * __uint_as_float(r[2 * j]), g * __uint_as_float(r[2 * j + 1]));
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(tb + lane * LDB + 16 * j) = pk[j];
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rl = i * 8 + rr;
                        if (q * 32 + rl < t.rows_valid)
                            *reinterpret_cast<uint4*>(out_h + ((long long)t.row0 + q * 32 + rl) * P.ld_out + t.out_col0 + c + cc * 8) =
                                *reinterpret_cast<const uint4*>(tb + rl * LDB + 16 * cc);
                    }
                    __syncwarp();
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) release_acc(acc);
            if (++acc == 2) {
                acc = 0;
                aph ^= 1u;
            }
        }
#ifdef DSMOE_TRACE
        GTRACE_ADD(5, t_all);
        if (warp == 2 && lane == 0 && blockIdx.x < 192) {
            long long* g = g_gemm_trace[P.epi == EPI_GELU ? 1 : (P.n_per_expert <= 192 ? 0 : 2)][blockIdx.x];
            g[5] = gtr[5];
            g[6] = gtr[6];
        }
#endif
    }

    // ---------------------------------------------------------------- teardown
teardown:
    ptx::tc_fence_before();
    if (PAIR) ptx::cluster_sync();      // neither CTA frees tensor memory or leaves while the other may still use or signal it
    else __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        if (PAIR) ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && P.dev_status) {
        if (sh.abort_flag) *P.dev_status = DSMOE_ERR_TIMEOUT;
        else if (sh.bad_offsets) *P.dev_status = DSMOE_ERR_INVALID_ARG;
    }
}

// ---------------------------------------------------------------- whole small-T layer in one launch
//
// Decode-sized calls are bound by reading the selected experts' weights once, and a 134 MB phase is
// too short to amortise a kernel launch, a prologue and a drained pipeline (about a quarter of its
// time).  So the whole layer runs as ONE cooperative launch of one CTA per SM.  All T <= 128 tokens
// ride in the one 128-row MMA tile, so the layer is evaluated in its gated dense form restricted to
// the experts that at least one token selected -- no grouping, no aggregation pass:
//
//   router   the reduction over d of every token cut into slices, one CTA each  -> grid barrier
//            every CTA adds every token's slices itself: softmax, selection (same arithmetic, same result
//            everywhere, so no second barrier); runs on the epilogue warps, underneath the up-projection
//   up       hg[t,(e,j)] = [e in sel(t)] S[t,e] GeLU(x[t].W1[e][:,j]); a CTA takes a contiguous run of
//            16-row units of the selected experts' W1 (a tile may cross one expert boundary) -> grid barrier
//   down     out = hg . W2cat as stream-K: units of (256 output columns, expert, 64-wide reduction
//            block); fp32 partial tiles, at most two per CTA                    -> grid barrier
//   fix-up   every CTA adds the partial tiles of its share of out[T,d] in ascending-CTA order
//
// From 8 tokens on the up-projection starts before the router has finished, under "every expert selected"
// (see the kernel).  The operand ring keeps running across the up/down barrier: the producer prefetches the
// first W2 tiles (which do not depend on hg) while other CTAs finish, asks the next ones into L2, and adds
// the hg tiles once the barrier has passed.  Every wait, on an mbarrier or on a grid barrier, is bounded.

struct SmallParams {
    int T, d, H, E, t_pad;
    const __nv_bfloat16* x;
    const float* Wr;
    const float* br;
    SelParams sel;
    float* scores;
    uint64_t* mask;
    int32_t* k_t;
    int32_t* counts_out;     // nullable
    __nv_bfloat16* hg;       // [T, E*H]
    float* partial;          // [grid][2][T][256]; doubles as the router's slice buffer
    void* out;
    int out_f32;
    int* sync;               // 8 ints, zero at launch: barrier counters [0..2] and an abort flag [4]
    int spec;                // start streaming under "every expert selected" before the router has finished
    int32_t* dev_status;
};

// One thread per CTA arrives at grid barrier `idx`; grid_wait spins (bounded) until all CTAs have.
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

struct SmallTile {
    int phase;                       // 0 up, 1 down
    int e, n0, bn, bn1, e2, nk;      // up: columns [0,bn1) are rows n0.. of expert e, [bn1,bn) rows 0.. of expert e2
    int out_col0, out_col0_2;
    int kstart, seg;                 // down: first global reduction block, partial-sum slot
};

struct SmallIter {
    int phase, u0, u1, r_first, down_u0, down_u1;

    int bn_down;

    // The two projections may be cut over different expert lists: the up-projection over n_up experts (all of
    // them, when it was started before the router had finished), the down-projection over the n_down selected ones.
    __device__ __forceinline__ void init(const SmallParams& P, int n_up, int n_down, int bn_down_) {
        const int G = gridDim.x;
        const int total = n_up * (P.H / kUpUnit);
        const int per = (total + G - 1) / G;
        u0 = min(total, (int)blockIdx.x * per);
        u1 = min(total, u0 + per);
        phase = 0;
        set_down(P, n_down, bn_down_);
    }
    __device__ __forceinline__ void set_down(const SmallParams& P, int n_down, int bn_down_) {
        const int G = gridDim.x;
        bn_down = bn_down_;
        const int U = n_down * (P.H / BK);
        const int total = ((P.d + bn_down - 1) / bn_down) * U;
        const int per = (total + G - 1) / G;
        down_u0 = min(total, (int)blockIdx.x * per);
        down_u1 = min(total, down_u0 + per);
        r_first = U > 0 ? down_u0 / U : 0;
    }
    // (re)start the down-projection under another expert list
    __device__ __forceinline__ void restart_down(const SmallParams& P, int n_down, int bn_down_) {
        set_down(P, n_down, bn_down_);
        phase = 1;
        u0 = down_u0;
        u1 = down_u1;
    }

    __device__ __forceinline__ bool next(const SmallParams& P, const int* active, int n_act, SmallTile& t) {
        if (phase == 0 && u0 >= u1) {
            phase = 1;
            u0 = down_u0;
            u1 = down_u1;
        }
        if (u0 >= u1) return false;
        t.phase = phase;
        t.e2 = 0;
        t.out_col0_2 = 0;
        t.kstart = 0;
        t.seg = 0;
        if (phase == 0) {
            const int upe = P.H / kUpUnit;
            const int ei = u0 / upe, in_e = u0 % upe;
            int len = min(u1 - u0, kUpTileUnits);
            const int len1 = min(len, upe - in_e);
            const int len2 = min(len - len1, upe);
            len = len1 + len2;
            t.e = active[ei];
            t.n0 = in_e * kUpUnit;
            t.bn1 = len1 * kUpUnit;
            t.bn = len * kUpUnit;
            t.nk = P.d / BK;
            t.out_col0 = t.e * P.H + t.n0;
            if (len2 > 0) {
                t.e2 = active[ei + 1];
                t.out_col0_2 = t.e2 * P.H;
            }
            u0 += len;
        } else {
            const int U = n_act * (P.H / BK);
            const int r = u0 / U, start = u0 % U;
            const int len = min(u1 - u0, U - start);
            t.e = 0;
            t.n0 = r * bn_down;
            t.bn = min(bn_down, P.d - t.n0);
            t.bn1 = t.bn;
            t.nk = len;
            t.kstart = start;
            t.seg = r - r_first;
            t.out_col0 = 0;
            u0 += len;
        }
        return true;
    }
};

// One ring slot's loads.  what: bit 0 = the token operand (x or hg), bit 1 = the weight rows.  The weights are read
// once per call, so their copies carry the evict-first L2 policy `wpol`: the stream then leaves the router's operands,
// hg, the partial sums and the kernel's own instructions in L2.
__device__ __forceinline__ void small_issue(const SmallParams& P, const CUtensorMap* tmX, const BMaps16* tmW1,
                                            const CUtensorMap* tmHg, const BMaps* tmW2, const int* active,
                                            const SmallTile& t, int i, uint32_t slotA, uint32_t slotB, uint32_t bar,
                                            int what, uint64_t wpol) {
    if (t.phase == 0) {
        if (what & 1) ptx::tma_load_2d(slotA, tmX, bar, i * BK, 0);
        if (what & 2) {
            ptx::tma_load_3d_hint(slotB, &tmW1->m[t.bn1 / 16 - 1], bar, 0, wrow(i, t.n0, P.H), t.e, wpol);
            if (t.bn > t.bn1)
                ptx::tma_load_3d_hint(slotB + t.bn1 * (BK * 2), &tmW1->m[(t.bn - t.bn1) / 16 - 1], bar, 0, wrow(i, 0, P.H), t.e2, wpol);
        }
    } else {
        const int kbpe = P.H / BK;
        const int g = t.kstart + i;
        const int e = active[g / kbpe], kb = g % kbpe;
        if (what & 1) ptx::tma_load_2d(slotA, tmHg, bar, e * P.H + kb * BK, 0);
        if (what & 2) {
            // column ranges are 64, 128 or 256 wide: one copy; only a ragged last range needs the decomposition
            if ((t.bn & (t.bn - 1)) == 0) ptx::tma_load_3d_hint(slotB, &tmW2->m[__ffs(t.bn) - 5], bar, 0, wrow(kb, t.n0, P.d), e, wpol);
            else load_weight_rows(tmW2, slotB, bar, wrow(kb, t.n0, P.d), t.bn, e);
        }
    }
}

// Ring geometry for n selected experts.  A slot holds the tokens' 64-wide block and one weight tile.  With few
// selected experts the tiles are narrow, so the down-projection takes narrower column ranges too and the ring
// has more slots: more loads in flight, which is what hides memory latency when each load is small.
__device__ __forceinline__ void small_geometry(const SmallParams& P, int n, int G, SmallGeo& g) {
    const int up_units = (n * (P.H / kUpUnit) + G - 1) / G;
    g.n_act = n;
    g.up_rows = max(1, min(up_units, kUpTileUnits)) * kUpUnit;
    g.bn_down = g.up_rows <= 64 ? 64 : g.up_rows <= 128 ? 128 : BN;
    g.a_bytes = P.t_pad * BK * 2;
    g.slot_bytes = g.a_bytes + g.bn_down * BK * 2;
    g.n_stages = max(2, min(MAX_STAGES, kSmallInflightBytes / g.slot_bytes));
}

// Second half of the router, run by the 12 epilogue warps of EVERY CTA: warp w owns tokens w, w + 12, ...; a lane
// holds experts lane and lane + 32.  Logits = bias plus the KS slice sums in ascending slice order, then softmax.
// The arithmetic is the same in every CTA, so are the results, and no grid barrier is needed to agree on them.
//   mode 0: selection -- sh.mask_s[token], sh.active_mask; CTA t also writes token t's scores, mask and count out
//   mode 1: router gates of experts e and e2 for every token (0 where not selected) -> sh.gate_s, sh.gate2_s
// KS * (tokens per warp) <= 16 for every T this kernel takes, so a warp fetches all its slice sums in one batch
// and waits for memory once.  One copy of this code serves both modes (not inlined): the second call finds its
// instructions cached, which matters while the weight stream keeps the memory system busy.
// What small_router_pass needs of the kernel's parameters, passed by value: a reference to the parameter block would
// make every thread copy all of it into local memory for the call.
struct RouterArgs {
    int T, E;
    const float* br;
    const float* partial;
    float* scores;
    uint64_t* mask;
    int32_t* k_t;
    SelParams sel;
};
__device__ __noinline__ void small_router_pass(const RouterArgs P, Shared& sh, int KS, int w, int lane, int mode, int e,
                                               int e2) {
    constexpr int NW = kEpiThreads / 32;
    if (KS == 0) {
        // One CTA per token held the whole reduction (KS = 1 in the kernel) and has written that token's scores and
        // selection itself before the grid barrier: here they are only read (a thread per token)
        const int tt = w * 32 + lane;
        if (mode == 0) {
            unsigned long long m = 0ull;
            if (tt < P.T) {
                m = __ldcg(reinterpret_cast<const unsigned long long*>(P.mask) + tt);
                sh.mask_s[tt] = m;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m |= __shfl_xor_sync(0xffffffffu, m, o);
            if (lane == 0 && m) atomicOr(&sh.active_mask, m);
        } else if (tt < P.T) {
            const uint64_t mk = sh.mask_s[tt];
            sh.gate_s[tt] = ((mk >> e) & 1ull) ? __ldcg(P.scores + (size_t)tt * P.E + e) : 0.f;
            sh.gate2_s[tt] = ((mk >> e2) & 1ull) ? __ldcg(P.scores + (size_t)tt * P.E + e2) : 0.f;
        }
        return;
    }
    const bool v_lo = lane < P.E, v_hi = lane + 32 < P.E;
    const float b_lo = (P.br && v_lo) ? P.br[lane] : 0.f, b_hi = (P.br && v_hi) ? P.br[lane + 32] : 0.f;
    const int ntok = w < P.T ? (P.T - w + NW - 1) / NW : 0;
    const int lg = 31 - __clz(KS);
    float vlo[16], vhi[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int tt = w + (j >> lg) * NW, sl = j & (KS - 1);      // KS is a power of two
        const bool ok = j < ntok * KS;
        const float* pl = P.partial + ((size_t)tt * KS + sl) * kMaxExperts;
        vlo[j] = (ok && v_lo) ? __ldcg(pl + lane) : 0.f;
        vhi[j] = (ok && v_hi) ? __ldcg(pl + lane + 32) : 0.f;
    }
#pragma unroll 1
    for (int i = 0; i < ntok; ++i) {
        const int tt = w + i * NW;
        float l_lo = b_lo, l_hi = b_hi;
#pragma unroll
        for (int j = 0; j < 16; ++j) {          // this token's slice sums are v[i KS .. i KS + KS): added in ascending order
            if ((j >> lg) == i) {
                l_lo += vlo[j];
                l_hi += vhi[j];
            }
        }
        float s_lo, s_hi;
        softmax_warp(l_lo, l_hi, P.E, lane, s_lo, s_hi);
        if (mode == 0) {
            const uint64_t m = select_warp(s_lo, s_hi, P.sel, lane);
            if (lane == 0) {
                sh.mask_s[tt] = m;
                atomicOr(&sh.active_mask, (unsigned long long)m);
            }
            if (tt == (int)blockIdx.x) {
                if (v_lo) P.scores[(size_t)tt * P.E + lane] = s_lo;
                if (v_hi) P.scores[(size_t)tt * P.E + lane + 32] = s_hi;
                if (lane == 0) {
                    P.mask[tt] = m;
                    if (P.k_t) P.k_t[tt] = __popcll(m);
                }
            }
        } else {
            const uint64_t mk = sh.mask_s[tt];
            if (lane == (e & 31)) sh.gate_s[tt] = ((mk >> e) & 1ull) ? (e < 32 ? s_lo : s_hi) : 0.f;
            if (lane == (e2 & 31)) sh.gate2_s[tt] = ((mk >> e2) & 1ull) ? (e2 < 32 ? s_lo : s_hi) : 0.f;
        }
    }
}

// Bounded wait for the router's verdict on the speculative geometry; 0 = gave up.
__device__ __forceinline__ int wait_geo(Shared& sh) {
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t spin = 0;; ++spin) {
        const int st = sh.geo_state;
        if (st) return st;
        if ((spin & 0xff) == 0xff) {
            if (sh.abort_flag) return 0;
            if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
                sh.abort_flag = 1;
                return 0;
            }
        }
    }
}
__device__ __forceinline__ bool wait_flag(volatile int* flag, Shared& sh) {
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t spin = 0;; ++spin) {
        if (*flag) return true;
        if ((spin & 0xff) == 0xff) {
            if (sh.abort_flag) return false;
            if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
                sh.abort_flag = 1;
                return false;
            }
        }
    }
}

__global__ void __launch_bounds__(SMALL_THREADS, 1)
small_layer_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ BMaps16 tmW1,
                   const __grid_constant__ CUtensorMap tmHg, const __grid_constant__ BMaps tmW2, const SmallParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw + (base - raw) + SMALL_RING_BYTES);
    float* stg = reinterpret_cast<float*>(smem_raw + (base - raw) + SMALL_RING_BYTES + SHARED_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_u32(&sh.tfull[a]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.tempty[a]), 4);
        }
        ptx::mbar_init(ptx::smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        sh.active_mask = 0ull;
        sh.geo_state = 0;
        sh.spec_issued = 0;
        sh.spec_stop = 0;
        sh.mma_drained = 0;
        sh.up_arrived = 0;
        small_geometry(P, P.E, G, sh.geo[0]);
#ifdef DSMOE_TRACE
        for (int i = 0; i < 32; ++i) sh.trace[i] = 0;
        TRACE(0);
#endif
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmX);
        ptx::prefetch_tensormap(&tmHg);
        ptx::prefetch_tensormap(&tmW1.m[sh.geo[0].up_rows / 16 - 1]);
        for (int i = 2; i < 5; ++i) ptx::prefetch_tensormap(&tmW2.m[i]);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    if (warp >= 2 && (int)threadIdx.x - 64 < kMaxExperts) sh.geo[0].active[threadIdx.x - 64] = (int)threadIdx.x - 64;
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;
    const uint32_t smA = base;

    // From here the three roles run side by side.  Warps 2.. compute the router (one grid barrier) and publish the
    // geometry it implies in geo[1]; warps 0 and 1 either wait for that, or (P.spec) start streaming and multiplying
    // the up-projection at once under geo[0], "every expert selected" -- the products x.W1 do not depend on the
    // router, only the partition of the work does.  If the router confirms geo[0] they simply carry on; if not,
    // the producer stops, the MMA issuer consumes what was loaded and waits for its products to retire, and both
    // start over under geo[1].  Ring slots keep one phase bit each (phb), so the ring may change its slot count
    // at that point without touching the barriers.
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t phb = 0;
            bool alive = true, spec = P.spec != 0;
            const uint64_t wpol = ptx::policy_evict_first();
            const SmallGeo* g = &sh.geo[0];
            if (!spec) {
                alive = wait_geo(sh) != 0;
                g = &sh.geo[1];
            }
            SmallIter it;
            SmallTile t;
            bool have = false;
            int n_stages = 1;
            uint32_t slot_bytes = 0, a_bytes = 0, smB = 0;
            for (int pass = 0; alive && pass < 2; ++pass) {
                n_stages = g->n_stages;
                slot_bytes = (uint32_t)g->slot_bytes;
                a_bytes = (uint32_t)g->a_bytes;
                smB = base + a_bytes;
                it.init(P, g->n_act, g->n_act, g->bn_down);
                have = it.next(P, g->active, g->n_act, t);
                int issued = 0;
                bool replaced = false;
                // up-projection
                while (alive && have && t.phase == 0 && !replaced) {
                    for (int i = 0; i < t.nk; ++i) {
                        const uint32_t ebar = ptx::smem_u32(&sh.empty[s]), epar = ((phb >> s) & 1u) ^ 1u;
                        if (spec) {
                            // the slot may never come back: once the router disagrees, the MMA issuer stops too
                            const uint64_t t0 = ptx::globaltimer_ns();
                            for (uint32_t spin = 1; !ptx::mbar_try_wait(ebar, epar); ++spin) {
                                if (sh.geo_state == 2) break;
                                if ((spin & 0xff) == 0 && (sh.abort_flag || ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs)) {
                                    sh.abort_flag = 1;
                                    alive = false;
                                    break;
                                }
                            }
                            if (!alive) break;
                            if (sh.geo_state == 2) {
                                replaced = true;
                                break;
                            }
                        } else if (!ptx::mbar_wait(ebar, epar, &sh.abort_flag)) {
                            alive = false;
                            break;
                        }
                        const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                        ptx::mbar_expect_tx(bar, a_bytes + (uint32_t)t.bn * BK * 2);
                        small_issue(P, &tmX, &tmW1, &tmHg, &tmW2, g->active, t, i, smA + s * slot_bytes, smB + s * slot_bytes, bar, 3, wpol);
                        phb ^= 1u << s;
                        ++issued;
                        if (++s == n_stages) s = 0;
                    }
                    if (!alive || replaced) break;
                    have = it.next(P, g->active, g->n_act, t);
                }
                if (alive && spec && !replaced) {
                    // the down-projection's partition needs the router's result
                    const int st = wait_geo(sh);
                    if (st == 0) alive = false;
                    else if (st == 2) replaced = true;
                    else {
                        g = &sh.geo[1];     // same ring; the down-projection runs over the selected experts
                        it.restart_down(P, g->n_act, g->bn_down);
                        have = it.next(P, g->active, g->n_act, t);
                    }
                }
                if (!(alive && replaced)) break;
                sh.spec_issued = issued;
                __threadfence_block();
                sh.spec_stop = 1;
                if (!wait_flag(&sh.mma_drained, sh)) alive = false;
                spec = false;
                g = &sh.geo[1];
                s = 0;
            }
            TRACE(3);
            // down-projection: weight tiles first, for as many slots as the ring has; their hg tiles follow
            // once every CTA has finished writing hg
            int pend_g[MAX_STAGES], pend_s[MAX_STAGES];      // reduction block and ring slot of each weight tile under way
            int npend = 0, i_cur = 0;
            while (alive && have && npend < n_stages) {
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ((phb >> s) & 1u) ^ 1u, &sh.abort_flag)) {
                    alive = false;
                    break;
                }
                const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                ptx::mbar_expect_tx(bar, a_bytes + (uint32_t)t.bn * BK * 2);
                small_issue(P, &tmX, &tmW1, &tmHg, &tmW2, g->active, t, i_cur, smA + s * slot_bytes, smB + s * slot_bytes, bar, 2, wpol);
                pend_g[npend] = t.kstart + i_cur;
                pend_s[npend] = s;
                ++npend;
                phb ^= 1u << s;
                if (++s == n_stages) s = 0;
                if (++i_cur == t.nk) {
                    i_cur = 0;
                    have = it.next(P, g->active, g->n_act, t);
                }
            }
            // Between the two projections HBM has nothing to do for several microseconds (epilogues, the slowest
            // CTA, the barrier), and the ring is full.  So the next weight tiles of this CTA's sequence are asked
            // into L2 meanwhile: the down-projection then finds them there instead of in DRAM.  All CTAs together
            // ask for well under half of L2.  (Not for the fewest tokens: there the gap is short and the requests only
            // compete with the ring's own.)
            if (alive && have && P.spec && wait_flag(&sh.up_arrived, sh)) {     // ... once this CTA's own hg is out
                SmallIter pit = it;
                SmallTile pt = t;
                int pi = i_cur;
                bool phave = have;
                const int kbpe = P.H / BK;
                for (int bytes = 0; phave && bytes < kSmallL2PrefetchBytes;) {
                    if ((pt.bn & (pt.bn - 1)) == 0) {
                        const int gb = pt.kstart + pi;
                        ptx::tma_prefetch_3d(&tmW2.m[__ffs(pt.bn) - 5], 0, wrow(gb % kbpe, pt.n0, P.d), g->active[gb / kbpe]);
                    }
                    bytes += pt.bn * BK * 2;
                    if (++pi == pt.nk) {
                        pi = 0;
                        phave = pit.next(P, g->active, g->n_act, pt);
                    }
                }
            }
            TRACE(5);
            if (alive && !grid_wait(P.sync, 1, G, &sh.abort_flag)) alive = false;
            TRACE(6);
            asm volatile("fence.proxy.async;" ::: "memory");   // hg was written through the generic proxy, TMA reads it
            for (int j = 0; alive && j < npend; ++j) {
                const int kbpe = P.H / BK, gb = pend_g[j];
                ptx::tma_load_2d(smA + pend_s[j] * slot_bytes, &tmHg, ptx::smem_u32(&sh.full[pend_s[j]]),
                                 g->active[gb / kbpe] * P.H + (gb % kbpe) * BK, 0);
            }
            while (alive && have) {
                for (; i_cur < t.nk; ++i_cur) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.empty[s]), ((phb >> s) & 1u) ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                    ptx::mbar_expect_tx(bar, a_bytes + (uint32_t)t.bn * BK * 2);
                    small_issue(P, &tmX, &tmW1, &tmHg, &tmW2, g->active, t, i_cur, smA + s * slot_bytes, smB + s * slot_bytes, bar, 3, wpol);
                    phb ^= 1u << s;
                    if (++s == n_stages) s = 0;
                }
                if (!alive) break;
                i_cur = 0;
                have = it.next(P, g->active, g->n_act, t);
            }
            if (!alive) {
                const uint64_t t0 = ptx::globaltimer_ns();   // copies already issued still land in this CTA's smem
                while (ptx::globaltimer_ns() - t0 < 200000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0, acc = 0;
            uint32_t phb = 0, aph = 0;
            bool alive = true, spec = P.spec != 0;
            const SmallGeo* g = &sh.geo[0];
            if (!spec) {
                alive = wait_geo(sh) != 0;
                g = &sh.geo[1];
            }
            for (int pass = 0; alive && pass < 2; ++pass) {
                const int n_stages = g->n_stages;
                const uint32_t slot_bytes = (uint32_t)g->slot_bytes, smB = base + (uint32_t)g->a_bytes;
                int consumed = 0;
                bool redo = false;
                SmallIter it;
                const SmallGeo* gD = g;      // the down-projection's expert list: geo[1] once the router is done
                it.init(P, g->n_act, g->n_act, g->bn_down);
                SmallTile t;
                for (;;) {
                    if (!(alive && !redo && it.next(P, g->active, gD->n_act, t))) {
                        if (alive && !redo && spec) {
                            // nothing (left) to do under geo[0]; there may be under geo[1], and if the router
                            // disagrees the producer waits for this thread
                            const int st = wait_geo(sh);
                            spec = false;
                            if (st == 0) alive = false;
                            else if (st == 2) redo = true;
                            else {
                                gD = &sh.geo[1];
                                it.restart_down(P, gD->n_act, gD->bn_down);
                                continue;
                            }
                        }
                        break;
                    }
                    if (spec && t.phase == 1) {
                        // no down-projection tile before the router has said over which experts it runs
                        const int st = wait_geo(sh);
                        if (st == 0) alive = false;
                        else if (st == 2) redo = true;
                        else {
                            spec = false;
                            gD = &sh.geo[1];
                            it.restart_down(P, gD->n_act, gD->bn_down);
                        }
                        continue;
                    }
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.tempty[acc]), aph ^ 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t idesc = ptx::make_idesc_bf16(BM, (uint32_t)t.bn);
                    const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                    for (int i = 0; i < t.nk; ++i) {
                        const uint32_t fbar = ptx::smem_u32(&sh.full[s]), par = (phb >> s) & 1u;
                        if (spec) {
                            // like mbar_wait, but the slot may never be filled: the producer stops when the router
                            // disagrees with the speculative geometry
                            const uint64_t t0 = ptx::globaltimer_ns();
                            for (uint32_t spin = 1; !ptx::mbar_try_wait(fbar, par); ++spin) {
                                if (sh.spec_stop && consumed == sh.spec_issued) {
                                    redo = true;
                                    break;
                                }
                                if ((spin & 0xff) == 0 && (sh.abort_flag || ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs)) {
                                    sh.abort_flag = 1;
                                    alive = false;
                                    break;
                                }
                            }
                            if (redo || !alive) break;
                        } else if (!ptx::mbar_wait(fbar, par, &sh.abort_flag)) {
                            alive = false;
                            break;
                        }
#ifdef DSMOE_TRACE
                        if (sh.trace[4] == 0) TRACE(4);
                        if (t.phase == 1 && sh.trace[8] == 0) TRACE(8);
                        if (t.phase == 0 && i < 8) TRACE(16 + i);
                        if (t.phase == 0 && i >= t.nk - 4) TRACE(24 + i - (t.nk - 4));
#endif
                        ptx::tc_fence_after();
                        // M = 128 although only t_pad rows were loaded: the rows beyond are whatever the ring holds,
                        // they only reach TMEM lanes that nobody reads
                        const uint32_t a0 = smA + s * slot_bytes, b0 = smB + s * slot_bytes;
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            ptx::umma_bf16(d_tmem, ptx::make_desc_k_sw128(a0 + k * 32), ptx::make_desc_k_sw128(b0 + k * 32),
                                           idesc, (uint32_t)((i | k) != 0));
                        ptx::umma_commit(ptx::smem_u32(&sh.empty[s]));
                        phb ^= 1u << s;
                        ++consumed;
                        if (++s == n_stages) s = 0;
                    }
                    if (!alive || redo) break;
                    if (spec) {
                        // a finished tile goes to the epilogue only once the router has confirmed its geometry
                        const int st = wait_geo(sh);
                        if (st == 0) {
                            alive = false;
                            break;
                        }
                        if (st == 2) {
                            redo = true;
                            break;
                        }
                        spec = false;
                        // the rest of the up-projection stays under geo[0]'s partition (and its identity expert list,
                        // which this thread's iterator already holds); the down-projection follows geo[1]
                        gD = &sh.geo[1];
                        it.set_down(P, gD->n_act, gD->bn_down);
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh.tfull[acc]));
                    if (++acc == 2) {
                        acc = 0;
                        aph ^= 1u;
                    }
                }
                if (!(alive && redo)) break;
                // take the remaining speculative loads off the ring, let the products issued so far retire, then
                // tell the producer that the ring is idle
                if (!wait_flag(&sh.spec_stop, sh)) break;
                const int issued = sh.spec_issued;
                while (alive && consumed < issued) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.full[s]), (phb >> s) & 1u, &sh.abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::mbar_arrive(ptx::smem_u32(&sh.empty[s]));
                    phb ^= 1u << s;
                    ++consumed;
                    if (++s == n_stages) s = 0;
                }
                if (!alive) break;
                ptx::umma_commit(ptx::smem_u32(&sh.drain));
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.drain), 0u, &sh.abort_flag)) break;
                __threadfence_block();
                sh.mma_drained = 1;
                spec = false;
                g = &sh.geo[1];
                s = 0;
                acc = 0;
                aph = 0;
            }
        }
    } else {
        // ------------------------------------------------------------ router, then epilogue (12 warps)
        const int etid = (int)threadIdx.x - 64;         // 0 .. kEpiThreads-1
#define EPI_SYNC() asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory")
        // ---- router, step 1
        // The reduction over d of every token is cut into KS slices, one CTA per (token, slice).  A row of Wr
        // (E floats) is covered by E/4 neighbouring threads with one 16-byte load each, so a warp reads whole
        // rows, coalesced, and a thread keeps only its four experts' sums over every rpp-th row; all its loads are
        // independent.  The threads' sums meet in shared memory.
        int KS = 1;                                   // 1, 2, 4, 8 or 16 slices
        while (KS < 16 && KS * 2 * P.T <= G) KS *= 2;
        if ((int)blockIdx.x < P.T * KS) {
            const int t = blockIdx.x / KS, sl = blockIdx.x % KS, E = P.E;
            const int klen = (P.d + KS - 1) / KS, kbeg = sl * klen, kend = min(P.d, kbeg + klen);
            const __nv_bfloat16* __restrict__ xr = P.x + (size_t)t * P.d;
            const float* __restrict__ Wr = P.Wr;
            const int quads = (E + 3) / 4;                  // threads per row
            const int rpp = kEpiThreads / quads;            // rows per pass
            const int qd = etid % quads, r0 = etid / quads;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            if (etid == 0) TRACE(12);
            if (r0 < rpp) {
                if ((E & 3) == 0) {
                    // batches of kRouterBatch rows: every load of a batch is issued before its first use
                    for (int kb = kbeg + r0; kb < kend; kb += kRouterBatch * rpp) {
                        float4 w[kRouterBatch];
                        float xs[kRouterBatch];
#pragma unroll
                        for (int j = 0; j < kRouterBatch; ++j) {
                            const int k = kb + j * rpp;
                            const bool ok = k < kend;
                            w[j] = ok ? __ldg(reinterpret_cast<const float4*>(Wr + (size_t)k * E) + qd) : make_float4(0.f, 0.f, 0.f, 0.f);
                            xs[j] = ok ? __bfloat162float(xr[k]) : 0.f;
                        }
#pragma unroll
                        for (int j = 0; j < kRouterBatch; ++j) {
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
                        const float* w = Wr + (size_t)k * E + e0;
                        acc.x = fmaf(xv, __ldg(w), acc.x);
                        if (e0 + 1 < E) acc.y = fmaf(xv, __ldg(w + 1), acc.y);
                        if (e0 + 2 < E) acc.z = fmaf(xv, __ldg(w + 2), acc.z);
                        if (e0 + 3 < E) acc.w = fmaf(xv, __ldg(w + 3), acc.w);
                    }
                }
            }
            if (etid == 0) TRACE(13);
            reinterpret_cast<float4*>(stg)[etid] = acc;      // stg[(r0 * quads + qd) * 4 + j]
            EPI_SYNC();
            if (etid < E) {
                const int e = etid;
                float v = 0.f;
                for (int r = 0; r < rpp; ++r) v += stg[(r * quads + (e >> 2)) * 4 + (e & 3)];
                P.partial[((size_t)t * KS + sl) * kMaxExperts + e] = v;   // the partial-sum buffer is free until the down-projection
                if (KS == 1) sh.gate_s[e] = v;          // the whole reduction: this CTA finishes its token below
            }
        }
        EPI_SYNC();
        // With one CTA per token (KS = 1: 37 tokens or more) the CTA holds its token's logits: it takes softmax and
        // selection itself and writes them out, and after the barrier every CTA reads all tokens' results instead of
        // repeating every token's softmax (at 128 tokens that repetition, once for the selection and once for the
        // gates, took 18 of the kernel's 76 us).  Same arithmetic as small_router_pass: bias + sum, softmax, selection.
        const bool direct = KS == 1;
        if (direct && (int)blockIdx.x < P.T && warp == 2) {
            const bool v_lo = lane < P.E, v_hi = lane + 32 < P.E;
            const float l_lo = v_lo ? (P.br ? P.br[lane] : 0.f) + sh.gate_s[lane] : 0.f;
            const float l_hi = v_hi ? (P.br ? P.br[lane + 32] : 0.f) + sh.gate_s[lane + 32] : 0.f;
            softmax_select_store(l_lo, l_hi, (int)blockIdx.x, P.sel, lane, P.scores, P.mask, P.k_t);
        }
        EPI_SYNC();
        if (etid == 0) {
            TRACE(1);
            grid_arrive(P.sync, 0);
            grid_wait(P.sync, 0, G, &sh.abort_flag);
            TRACE(14);
        }
        EPI_SYNC();
        // ---- router, step 2: softmax and selection of every token, in every CTA (see small_router_pass)
        const RouterArgs RA{P.T, P.E, P.br, P.partial, P.scores, P.mask, P.k_t, P.sel};
        if (!sh.abort_flag) small_router_pass(RA, sh, direct ? 0 : KS, warp - 2, lane, 0, 0, 0);
        EPI_SYNC();
        if (etid == 0) {
            unsigned long long m = sh.active_mask;
            if (P.E < 64) m &= (1ull << P.E) - 1ull;
            SmallGeo& gr = sh.geo[1];
            int n = 0;
            for (int e = 0; e < P.E; ++e)
                if ((m >> e) & 1ull) gr.active[n++] = e;
            small_geometry(P, n, G, gr);
            // an up-projection already under way stands if at most an eighth of the experts went unselected (and
            // the ring keeps its geometry): starting over would cost more than their tiles do
            const SmallGeo& g0 = sh.geo[0];
            const bool keep = P.spec && (n == P.E || (n >= P.E - max(1, P.E / 8) && gr.a_bytes == g0.a_bytes &&
                                                      gr.slot_bytes == g0.slot_bytes && gr.n_stages == g0.n_stages));
            if (!keep) ptx::prefetch_tensormap(&tmW1.m[gr.up_rows / 16 - 1]);
            sh.up_geo = keep ? 0 : 1;
            __threadfence_block();
            sh.geo_state = keep ? 1 : 2;
            TRACE(2);
        }
        EPI_SYNC();
        const SmallGeo& ge = sh.geo[1];
        const SmallGeo& gu = sh.geo[sh.up_geo];
        const int n_act = ge.n_act;
        const bool aborted_early = sh.abort_flag != 0;

        // ---- epilogue
        const int q = warp & 3;
        const bool tmem_warp = warp < 6;                 // warps 2..5 read TMEM; warps 6.. only share the arithmetic
        int acc = 0;
        uint32_t aph = 0;
        bool dead = aborted_early;     // a dead warp still takes part in every named barrier below
        bool up_done = false;
        SmallIter it;
        it.init(P, gu.n_act, n_act, ge.bn_down);
        SmallTile t;
        const int row = q * 32 + lane;
        for (;;) {
            const bool have = it.next(P, gu.active, n_act, t);
            if (!up_done && (!have || t.phase == 1)) {
                // this CTA's part of hg is complete: publish it (the arriving thread's fence, after the barrier,
                // covers the other threads' stores), then signal the up/down grid barrier
                asm volatile("fence.proxy.async;" ::: "memory");
                EPI_SYNC();
                if (etid == 0) {
                    grid_arrive(P.sync, 1);
                    sh.up_arrived = 1;
                    TRACE(7);
                }
                up_done = true;
            }
            if (!have) break;
            // router gate of every token for this tile's expert(s), recomputed from the slice sums (other CTAs' copies
            // of the scores are not visible yet) while the mainloop is still running
            if (t.phase == 0 && !dead) small_router_pass(RA, sh, direct ? 0 : KS, warp - 2, lane, 1, t.e, t.e2);
            if (tmem_warp && !dead && !ptx::mbar_wait(ptx::smem_u32(&sh.tfull[acc]), aph, &sh.abort_flag)) dead = true;
            dead = __any_sync(0xffffffffu, dead);     // the TMEM reads below are warp-collective
#ifdef DSMOE_TRACE
            if (etid == 0 && t.phase == 0) TRACE(28);
#endif
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t)(acc * BN) + ((uint32_t)(q * 32) << 16);
            if (t.phase == 0) {
                // Few tokens fill only the first TMEM lanes, so one warp would do all the GeLU work.  Instead the
                // warps that own valid lanes copy the accumulators to shared memory, as many columns per round as the
                // staging tile holds for T rows, and all 128 epilogue threads share the arithmetic.
                // columns per round: what the staging tile holds for T rows (a power of two, at most a whole tile)
                constexpr int kStgFloats = STG_BYTES / 4;
                int CH = 256;
                while (CH > 32 && P.T * (CH + 4) > kStgFloats) CH >>= 1;
                const int ld = CH + 4;                                                    // floats per staged row
                for (int c0 = 0; c0 < t.bn; c0 += CH) {
                    const int cw = min(CH, t.bn - c0);
                    if (tmem_warp && !dead && q * 32 < P.T) {
                        for (int c = 0; c < cw; c += 32) {
                            uint32_t r[32];
                            ptx::tmem_ld32(taddr + (uint32_t)(c0 + c), r);
                            ptx::tmem_ld_wait();
                            if (row < P.T) {
                                float4* dst = reinterpret_cast<float4*>(stg + row * ld + c);
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                         __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                            }
                        }
                    }
                    EPI_SYNC();
#ifdef DSMOE_TRACE
                    if (etid == 0) TRACE(29 + (c0 > 0));
#endif
                    const int groups = cw / 8;
                    const int items = P.T * groups;
                    for (int item = etid; !dead && item < items; item += kEpiThreads) {
                        const int rr = item / groups, cg = item % groups;
                        const float4 a = *reinterpret_cast<const float4*>(stg + rr * ld + cg * 8);
                        const float4 b = *reinterpret_cast<const float4*>(stg + rr * ld + cg * 8 + 4);
                        const int col = c0 + cg * 8;           // 8-column groups never straddle the expert boundary
                        const bool second = col >= t.bn1;
                        const float g = second ? sh.gate2_s[rr] : sh.gate_s[rr];
                        const long long ocol = second ? (long long)t.out_col0_2 + (col - t.bn1) : (long long)t.out_col0 + col;
                        uint4 pk;
                        __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&pk);
                        hv[0] = __floats2bfloat162_rn(g * gelu_erf(a.x), g * gelu_erf(a.y));
                        hv[1] = __floats2bfloat162_rn(g * gelu_erf(a.z), g * gelu_erf(a.w));
                        hv[2] = __floats2bfloat162_rn(g * gelu_erf(b.x), g * gelu_erf(b.y));
                        hv[3] = __floats2bfloat162_rn(g * gelu_erf(b.z), g * gelu_erf(b.w));
                        *reinterpret_cast<uint4*>(P.hg + (long long)rr * ((long long)P.E * P.H) + ocol) = pk;
                    }
                    EPI_SYNC();
                }
            } else {
                // fp32 partial sums of this CTA's share of the reduction: slot (cta, seg), row, 256 columns
                for (int c = 0; tmem_warp && !dead && q * 32 < P.T && c < t.bn; c += 32) {
                    uint32_t r[32];
                    ptx::tmem_ld32(taddr + (uint32_t)c, r);
                    ptx::tmem_ld_wait();
                    if (row < P.T) {
                        float4* dst = reinterpret_cast<float4*>(P.partial + (((long long)blockIdx.x * 2 + t.seg) * P.T + row) * BN + c);
                        const int ncol = min(32, t.bn - c);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (j * 4 < ncol)
                                dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                     __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (tmem_warp && lane == 0 && !dead) ptx::mbar_arrive(ptx::smem_u32(&sh.tempty[acc]));
            if (++acc == 2) {
                acc = 0;
                aph ^= 1u;
            }
        }
        // ---- last grid barrier, then the fix-up: out[t,c] = sum of the partial tiles covering column c in
        // ascending CTA order (the partition arithmetic mirrors SmallIter).  The arriving thread's fence, after
        // the CTA barrier, covers the other threads' partial-sum stores.
        EPI_SYNC();
        if (etid == 0) {
            TRACE(9);
            grid_arrive(P.sync, 2);
            if (!grid_wait(P.sync, 2, G, &sh.abort_flag)) sh.abort_flag = 1;
            TRACE(10);
        }
        EPI_SYNC();
        if (!sh.abort_flag) {
            const int kbpe = P.H / BK;
            const int U = n_act * kbpe;
            const int bnd = ge.bn_down;
            const int nr = (P.d + bnd - 1) / bnd;
            const int total = nr * U;
            const int per = total > 0 ? (total + G - 1) / G : 1;
            // a thread owns 4 consecutive columns of one token; its partial loads are issued in batches before
            // the additions, which run in ascending CTA order
            const int d4 = P.d / 4;
            const int n_out4 = P.T * d4;                        // T <= 128 and d < 2^16: an int
            const int per_cta = (n_out4 + G - 1) / G;           // an equal share for every CTA
            for (int j = etid; j < per_cta; j += kEpiThreads) {
                const int idx = (int)blockIdx.x * per_cta + j;
                if (idx >= n_out4) break;
                const int tt = idx / d4, col = (idx % d4) * 4;
                const int r = col / bnd, cc = col % bnd;
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                if (U > 0) {
                    const int i0 = (r * U) / per, i1 = ((r + 1) * U - 1) / per;
                    // CTA i0 may have started in the range before (then range r is its second one); every later
                    // contributor starts inside range r
                    const int seg_first = i0 * per < r * U ? 1 : 0;
                    for (int ib = i0; ib <= i1; ib += kFixBatch) {
                        float4 v[kFixBatch];
#pragma unroll
                        for (int j = 0; j < kFixBatch; ++j) {
                            const int i = ib + j;
                            const int seg = i == i0 ? seg_first : 0;
                            v[j] = i <= i1 ? __ldcg(reinterpret_cast<const float4*>(
                                                 P.partial + (((long long)i * 2 + seg) * P.T + tt) * BN + cc))
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int j = 0; j < kFixBatch; ++j) {
                            sum.x += v[j].x;
                            sum.y += v[j].y;
                            sum.z += v[j].z;
                            sum.w += v[j].w;
                        }
                    }
                }
                if (P.out_f32) {
                    reinterpret_cast<float4*>(P.out)[idx] = sum;
                } else {
                    uint2 pk;
                    *reinterpret_cast<__nv_bfloat162*>(&pk.x) = __floats2bfloat162_rn(sum.x, sum.y);
                    *reinterpret_cast<__nv_bfloat162*>(&pk.y) = __floats2bfloat162_rn(sum.z, sum.w);
                    reinterpret_cast<uint2*>(P.out)[idx] = pk;
                }
            }
            if (P.counts_out && blockIdx.x == 0 && etid < P.E) {
                int n = 0;
                for (int tt = 0; tt < P.T; ++tt) n += (int)((sh.mask_s[tt] >> etid) & 1ull);
                P.counts_out[etid] = n;
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
#ifdef DSMOE_TRACE
    if (threadIdx.x == 0 && blockIdx.x < 192) {
        TRACE(11);
        for (int i = 0; i < 32; ++i) g_trace[blockIdx.x][i] = sh.trace[i];
    }
#endif
    if (threadIdx.x == 0 && sh.abort_flag) {
        atomicExch(P.sync + 4, 1);
        if (P.dev_status) *P.dev_status = DSMOE_ERR_TIMEOUT;
    }
}

// ---------------------------------------------------------------- host side

// DSMOE_GEMM_PAIR=0 in the environment keeps umma_gemm_kernel to single CTAs, =1 pairs wherever the shapes allow
// (tuning aid); unset, launch_gemm decides.
int pair_override() {
    const char* e = getenv("DSMOE_GEMM_PAIR");     // read at every launch: a test switches it between calls
    return e && *e ? atoi(e) : -1;
}

// pair_tiles: an upper bound of the number of 256-row tiles (INT_MAX where only the device knows, as in the grouped
// modes); 0 = never pair (the caller's shapes do not allow it).
dsmoe_status launch_gemm(const CUtensorMap& a, const BMaps& b, const GemmParams& P_in, int grid, cudaStream_t s,
                         bool may_time = true, int pair_tiles = 0) {
    DeviceState* st = nullptr;
    DSMOE_TRY(device_state(&st));
    if (!st->attr_gemm) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(umma_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_GEMM_CMB_BYTES));
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(umma_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_GEMM_CMB_BYTES));
        st->attr_gemm = true;
    }
    const GemmParams& P = P_in;
    int threads = (P.gather || P.epi == EPI_COMBINE) ? GATHER_THREADS : NUM_THREADS;
    // the ring, the barriers, and the tiles the epilogues send their rows through
    const size_t smem = SMEM_GEMM_CMB_BYTES;
    if (st->max_pairs < 0) {
        // how many clusters of two CTAs fit the device at once (the persistent kernel launches no more)
        cudaLaunchConfig_t q{};
        q.gridDim = dim3(2 * (st->sm_count / 2));
        q.blockDim = dim3(GATHER_THREADS);
        q.dynamicSmemBytes = SMEM_GEMM_CMB_BYTES;
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
        q.attrs = qa; q.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, umma_gemm_kernel<true>, &q) != cudaSuccess) {
            cudaGetLastError();
            n = 0;
        }
        st->max_pairs = n < st->sm_count / 2 ? n : st->sm_count / 2;
    }
    // Measured (C3, C4 and the paper's shapes): pairs gain 3 to 8 % where a long mainloop runs against a light
    // epilogue (plain stores after a reduction of 1024 or more), lose up to 9 % under the GeLU and gathering
    // up-projections and on short reductions, and change nothing under the aggregating epilogue.
    bool pair = pair_tiles > 0 && st->max_pairs > 0 && (P.n_per_expert % 64) == 0;
    if (pair_override() == 0) pair = false;
    else if (pair && pair_override() != 1)
        pair = P.epi == EPI_STORE && pair_tiles >= st->max_pairs && (P.mode == GEMM_DENSE_DOWN || P.k_per_expert >= 1024);
    int timed = -1;
    if (may_time) DSMOE_TRY(timing_begin(s, &timed));
    if (pair) {
        if (P.gather) threads = NUM_THREADS + 32 * Geo<true>::GW;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(2 * (pair_tiles < st->max_pairs ? pair_tiles : st->max_pairs));
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        int na = 1;
        if (P.epi == EPI_COMBINE) {      // its epilogues wait for one another's tiles: every CTA must be resident
            at[na].id = cudaLaunchAttributeCooperative;
            at[na].val.cooperative = 1;
            ++na;
        }
        cfg.attrs = at; cfg.numAttrs = na;
        DSMOE_CUDA_TRY(cudaLaunchKernelEx(&cfg, umma_gemm_kernel<true>, a, b, P));
    } else if (P.epi == EPI_COMBINE) {
        // its epilogues wait for one another's tiles: every CTA must be resident
        void* args[] = {const_cast<CUtensorMap*>(&a), const_cast<BMaps*>(&b), const_cast<GemmParams*>(&P)};
        DSMOE_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(umma_gemm_kernel<false>), dim3(grid), dim3(threads),
                                                   args, smem, s));
    } else {
        umma_gemm_kernel<false><<<grid, threads, smem, s>>>(a, b, P);
        DSMOE_CUDA_TRY(cudaGetLastError());
    }
    DSMOE_TRY(timing_end(s, timed));
    return DSMOE_OK;
}

// ---------------------------------------------------------------- router logits on the tensor cores
// Wr (fp32) is written as the exact sum of three bf16 terms, w = w1 + w2 + w3 (w1 = bf16(w), w2 = bf16(w - w1),
// w3 = bf16(w - w1 - w2): 3 x 8 significant bits cover fp32's 24).  x is bf16, so every product x.w_i is exact in
// fp32 and the three sums accumulate in fp32: the logits are as accurate as an fp32 dot product, at tensor-core
// speed.  The three terms sit side by side along N: B = [3 * EP, d] bf16 in the packed weights' layout, EP = E rounded up to 32 or 64.
__global__ void __launch_bounds__(256) router_split_kernel(const float* __restrict__ Wr, __nv_bfloat16* __restrict__ out,
                                                           int d, int E, int EP) {
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (long long)EP * d) return;
    const int e = (int)(idx / d), k = (int)(idx % d);
    const float w = e < E ? Wr[(size_t)k * E + e] : 0.f;
    const __nv_bfloat16 w1 = __float2bfloat16_rn(w);
    const float r1 = w - __bfloat162float(w1);
    const __nv_bfloat16 w2 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(w2);
    // block-major like the packed expert weights: [k / 64][3 * EP][64], term g in rows g * EP .. of every block
    const long long o = ((long long)(k / BK) * (3 * EP) + e) * BK + k % BK;
    out[o] = w1;
    out[o + (long long)EP * BK] = w2;
    out[o + 2ll * EP * BK] = __float2bfloat16_rn(r2);
}

// logits = (s1 + s2) + s3 + bias per expert, then softmax and selection: one warp per token
// (the reduction over d may come in `pieces` blocks of 3 EP sums each, added in ascending order).  A block is one
// chunk of 32 tokens; with chunk_counts its first warp then counts, per expert, the chunk's tokens that selected it
// (what chunk_count_kernel would write to chunk_prefix[chunk,:]).
__global__ void __launch_bounds__(32 * kChunk, 2) router_finish_kernel(const float* __restrict__ sums, const float* __restrict__ br,
                                                                    float* __restrict__ scores, uint64_t* __restrict__ mask,
                                                                    int32_t* __restrict__ k_t, int32_t* __restrict__ chunk_counts,
                                                                    int T, int EP, int pieces, SelParams q) {
    __shared__ uint64_t mask_s[kChunk];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * kChunk + warp;
    uint64_t m = 0;
    if (t < T) {
        const float* row = sums + (size_t)t * 3 * EP * pieces;
        const bool v_lo = lane < q.E, v_hi = lane + 32 < q.E;
        float l_lo = 0.f, l_hi = 0.f;
        for (int pc = 0; pc < pieces; ++pc, row += 3 * EP) {
            if (v_lo) l_lo += (row[lane] + row[EP + lane]) + row[2 * EP + lane];
            if (v_hi) l_hi += (row[lane + 32] + row[EP + lane + 32]) + row[2 * EP + lane + 32];
        }
        if (v_lo && br) l_lo += br[lane];
        if (v_hi && br) l_hi += br[lane + 32];
        m = softmax_select_store(l_lo, l_hi, t, q, lane, scores, mask, k_t);
    }
    if (!chunk_counts) return;
    if (lane == 0) mask_s[warp] = m;
    __syncthreads();
    if (warp == 0) {
        const uint64_t mt = mask_s[lane];
        int c_lo = 0, c_hi = 0;
        for (int e = 0; e < q.E; ++e) {
            const int n = __popc(__ballot_sync(0xffffffffu, (mt >> e) & 1));
            if (lane == (e & 31)) {
                if (e < 32) c_lo = n; else c_hi = n;
            }
        }
        if (lane < q.E) chunk_counts[(size_t)blockIdx.x * q.E + lane] = c_lo;
        if (lane + 32 < q.E) chunk_counts[(size_t)blockIdx.x * q.E + lane + 32] = c_hi;
    }
}

// out[r,:] (bf16) = the sum over the splits, in ascending order, of the fp32 partial rows part[s * split_rows + r,:]
// that a launch with k_splits left behind; rows from offsets[E] on do not exist
__global__ void __launch_bounds__(256) split_sum_kernel(const float4* __restrict__ part, int splits, int split_rows,
                                                        const int32_t* __restrict__ offsets, int E, int n,
                                                        __nv_bfloat16* __restrict__ out) {
    const int nvec = n / 4;
    const long long rows = min(max(offsets[E], 0), split_rows);
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < rows * nvec; i += (long long)gridDim.x * 256) {
        float4 a = part[i];
        for (int sp = 1; sp < splits; ++sp) {
            const float4 b = part[(long long)sp * split_rows * nvec + i];
            a.x += b.x;
            a.y += b.y;
            a.z += b.z;
            a.w += b.w;
        }
        uint2 pk;
        *reinterpret_cast<__nv_bfloat162*>(&pk.x) = __floats2bfloat162_rn(a.x, a.y);
        *reinterpret_cast<__nv_bfloat162*>(&pk.y) = __floats2bfloat162_rn(a.z, a.w);
        reinterpret_cast<uint2*>(out)[i] = pk;
    }
}

}  // namespace

// With few row tiles the logits' reduction over d is cut into 2 or 4 pieces, each a tile with its own block of sums,
// so that the launch covers most SMs instead of T / 128 of them.
constexpr int kRouterMaxPieces = 4;

size_t router_umma_scratch(const dsmoe_layer_desc& p, size_t* split_bytes) {
    const size_t EP = p.E <= 32 ? 32 : 64;
    const size_t a = align_up(3 * EP * (size_t)p.d * 2, 256);
    if (split_bytes) *split_bytes = a;
    return a + align_up((size_t)p.T * kRouterMaxPieces * 3 * EP * 4, 256);
}

bool router_umma_supported(const dsmoe_layer_desc& p) { return umma_supported(p) && p.T > 256; }

dsmoe_status launch_router_umma(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                float* scores, uint64_t* mask, int32_t* k_t, char* scratch, int32_t* dev_status,
                                cudaStream_t s, int32_t* chunk_counts) {
    const int EP = p.E <= 32 ? 32 : 64;
    size_t split_bytes = 0;
    router_umma_scratch(p, &split_bytes);
    __nv_bfloat16* wsplit = reinterpret_cast<__nv_bfloat16*>(scratch);
    float* sums = reinterpret_cast<float*>(scratch + split_bytes);
    router_split_kernel<<<ceil_div(EP * p.d, 256), 256, 0, s>>>(Wr, wsplit, p.d, p.E, EP);
    DSMOE_CUDA_TRY(cudaGetLastError());
    const CUtensorMap* mA;
    const BMaps* mB;
    DSMOE_TRY(cached_map_2d(&mA, x, p.T, p.d, BM));
    const int row_tiles = ceil_div(p.T, BM);
    int pieces = kRouterMaxPieces;
    while (pieces > 1 && (row_tiles * pieces > sm_count() || (p.d / BK) % pieces)) pieces /= 2;
    DSMOE_TRY(cached_bmaps(&mB, wsplit, pieces, 3 * EP, p.d / pieces));
    GemmParams g{};
    g.mode = GEMM_DENSE_UP; g.epi = EPI_STORE; g.E = pieces; g.n_per_expert = 3 * EP; g.k_per_expert = p.d / pieces;
    g.a_expert_stride = p.d / pieces; g.rows = p.T;
    g.out = sums; g.ld_out = (long long)pieces * 3 * EP; g.out_f32 = 1; g.dev_status = dev_status;
    const int tiles = row_tiles * pieces;
    DSMOE_TRY(launch_gemm(*mA, *mB, g, tiles < sm_count() ? tiles : sm_count(), s, false));
    router_finish_kernel<<<ceil_div(p.T, kChunk), 32 * kChunk, 0, s>>>(sums, br, scores, mask, k_t, chunk_counts, p.T, EP, pieces,
                                                         SelParams{p.E, p.mode, p.eps, p.eps_normalized, p.K, p.min_k, nullptr});
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

#ifdef DSMOE_TRACE
extern "C" __attribute__((visibility("default"))) int dsmoe_trace_read(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_trace, sizeof(unsigned long long) * 192 * 32);
}
extern "C" __attribute__((visibility("default"))) int dsmoe_gemm_trace_read(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_gemm_trace, sizeof(long long) * 3 * 192 * 8);
}
#endif

bool umma_supported(const dsmoe_layer_desc& p) {
    return p.dtype == DSMOE_BF16 && (p.d % 64) == 0 && (p.H % 64) == 0;
}

dsmoe_status launch_mlp_umma(const dsmoe_layer_desc& p, const void* xp, const void* packed, const int32_t* offsets,
                             void* hbuf, void* yp, int32_t* dev_status, cudaStream_t s, const void* x,
                             const int32_t* row_token, const CombineArgs* cmb, const MoaCore* moa) {
    if (p.T == 0) return DSMOE_OK;
    if (!umma_supported(p)) return DSMOE_ERR_UNSUPPORTED;
    const size_t amax = amax_of(p);
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    const CUtensorMap *mA1, *mA2;
    const BMaps *mB1, *mB2;
    // with row_token, the up-projection fetches its rows straight from x (no grouped copy of the tokens); its A
    // tensor map is then unused, any valid one will do
    DSMOE_TRY(cached_map_2d(&mA1, row_token ? hbuf : xp, amax, row_token ? p.H : p.d, BM));
    DSMOE_TRY(cached_bmaps(&mB1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_map_2d(&mA2, hbuf, amax, p.H, BM));
    DSMOE_TRY(cached_bmaps(&mB2, w2t, p.E, p.d, p.H));
    GemmParams up{};
    up.mode = GEMM_GROUPED; up.epi = EPI_GELU; up.E = p.E; up.n_per_expert = p.H; up.k_per_expert = p.d;
    up.rows = (int)amax; up.offsets = offsets; up.out = hbuf; up.ld_out = p.H; up.dev_status = dev_status;
    up.gather = row_token;
    up.gather_src = x;
    up.gather_rows = p.T;
    if (moa) up.epi = EPI_STORE;      // query projection: no activation (Eq. 7)
    GemmParams down{};
    down.mode = GEMM_GROUPED; down.epi = EPI_STORE; down.E = p.E; down.n_per_expert = p.d; down.k_per_expert = p.H;
    down.rows = (int)amax; down.offsets = offsets; down.out = yp; down.ld_out = p.d; down.dev_status = dev_status;
    if (cmb && !cmb->out) {
        down.row_gate = cmb->row_gate;     // yp[r,:] = gate[r] * (h.W2[e])[r,:] in fp32: no rounding before the sum
        down.out_f32 = 1;
    } else if (cmb) {
        // Eq. 1's weighted sum inside the down-projection's epilogue: no expert-output buffer, no aggregation pass
        down.epi = EPI_COMBINE;
        down.out = cmb->out;
        down.out_f32 = p.out_fp32 ? 1 : 0;
        down.row_token = cmb->row_token;
        down.row_gate = cmb->row_gate;
        down.sel_mask = cmb->mask;
        down.acc = p.out_fp32 ? static_cast<float*>(cmb->out) : cmb->acc;
        down.tile_done = cmb->tile_done;
        down.tokens = p.T;
        DSMOE_CUDA_TRY(cudaMemsetAsync(cmb->tile_done, 0, (size_t)p.E * ceil_div(p.d, BN) * sizeof(int), s));
    }
    // 256-row tiles (CTA pairs) waste little only where experts hold many rows; the host knows their number for a
    // top-K selection alone (an upper bound otherwise), so only there may the launches pair on their own
    const long long known = p.mode == DSMOE_SELECT_TOPK ? (long long)p.T * (p.K < p.E ? p.K : p.E) : 0;
    const int pair_tiles = known >= 1024ll * p.E ? INT_MAX : (pair_override() == 1 ? INT_MAX : 0);
    // Few rows and a long reduction (the query projection at decode sizes: a handful of tiles, each a chain of d / 64
    // reduction blocks): the reduction is cut so that the launch covers the SMs; the partial sums (fp32, in the buffer
    // of the expert outputs, which is idle until the output projection) are added in order by split_sum_kernel
    int splits = 1;
    if (moa && yp && cmb && !cmb->out) {
        const long long max_tiles = ((long long)(amax / BM) + p.E) * ceil_div(p.H, BN);
        while (splits < 8 && max_tiles * splits * 2 <= sm_count() && (p.d / BK) % (splits * 2) == 0 &&
               (p.d / BK) / (splits * 2) >= 4 && (long long)splits * 2 * p.H <= p.d)
            splits *= 2;
    }
    if (splits > 1) {
        up.k_splits = splits; up.split_rows = (int)amax;
        up.out = yp; up.out_f32 = 1;
        DSMOE_TRY(launch_gemm(*mA1, *mB1, up, sm_count(), s, true, 0));
        const long long vecs = (long long)amax * p.H / 4;
        split_sum_kernel<<<(int)std::min<long long>((vecs + 255) / 256, 8ll * sm_count()), 256, 0, s>>>(
            static_cast<const float4*>(yp), splits, (int)amax, offsets, p.E, p.H, static_cast<__nv_bfloat16*>(hbuf));
        DSMOE_CUDA_TRY(cudaGetLastError());
    } else {
        DSMOE_TRY(launch_gemm(*mA1, *mB1, up, sm_count(), s, true, moa ? 0 : pair_tiles));
    }
    if (moa) DSMOE_TRY(launch_moa_attention(p, *moa, hbuf, row_token, moa->token_rows, offsets, dev_status, s));
    DSMOE_TRY(launch_gemm(*mA2, *mB2, down, sm_count(), s, true, pair_tiles));
    return DSMOE_OK;
}

// Few tokens (decode): one cooperative launch of small_layer_kernel runs router, both projections and the
// fix-up.
bool small_supported(const dsmoe_layer_desc& p) {
    const int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    if (!(umma_supported(p) && p.T >= 1 && p.T <= kSmallMaxT && p.T <= G && ceil_div(p.d, 64) <= G)) return false;
    if (p.mode == DSMOE_SELECT_THRESHOLD_TOPK) return false;   // its K needs a pass over the batch first: grouped path
    // the router's second half fetches all slice sums of a warp's tokens in one batch of 16 (small_router_pass)
    int KS = 1;
    while (KS < 16 && KS * 2 * p.T <= G) KS *= 2;
    return KS * ceil_div(p.T, kEpiThreads / 32) <= 16;
}

dsmoe_status launch_layer_small(const dsmoe_layer_desc& p, const void* x, const float* Wr, const float* br,
                                const void* packed, float* scores, uint64_t* mask, int32_t* k_t, int32_t* counts_out,
                                void* out, char* ws, const WsLayout& L, int32_t* dev_status, cudaStream_t s) {
    DeviceState* st = nullptr;
    DSMOE_TRY(device_state(&st));
    if (!st->attr_small) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(small_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
        st->attr_small = true;
    }
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    const int t_pad = (p.T + 7) / 8 * 8;
    int G = sm_count() < kSmallMaxCtas ? sm_count() : kSmallMaxCtas;
    void* hg = ws + L.h;
    const CUtensorMap *mX, *mHg;
    const BMaps16* mW1;
    const BMaps* mW2;
    DSMOE_TRY(cached_map_2d(&mX, x, p.T, p.d, t_pad));
    DSMOE_TRY(cached_bmaps16(&mW1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_map_2d(&mHg, hg, p.T, (uint64_t)p.E * p.H, t_pad));
    DSMOE_TRY(cached_bmaps(&mW2, w2t, p.E, p.d, p.H));
    SmallParams P;
    P.T = p.T; P.d = p.d; P.H = p.H; P.E = p.E; P.t_pad = t_pad;
    P.x = static_cast<const __nv_bfloat16*>(x);
    P.Wr = Wr;
    P.br = br;
    P.sel = SelParams{p.E, p.mode, p.eps, p.eps_normalized, p.K, p.min_k, nullptr};
    P.scores = scores;
    P.mask = mask;
    P.k_t = k_t;
    P.counts_out = counts_out;
    P.hg = static_cast<__nv_bfloat16*>(hg);
    P.partial = reinterpret_cast<float*>(ws + L.partial);
    P.out = out;
    P.out_f32 = p.out_fp32 ? 1 : 0;
    P.sync = reinterpret_cast<int*>(ws + L.sync);
    P.dev_status = dev_status;
    // From kSpecMinT tokens on it is rare that an expert is selected by none of them, so the kernel starts the
    // up-projection under that assumption while its router is still running; it starts over if the router disagrees.
    P.spec = p.T >= kSpecMinT ? 1 : 0;
    DSMOE_CUDA_TRY(cudaMemsetAsync(P.sync, 0, 32, s));
    void* args[] = {const_cast<CUtensorMap*>(mX), const_cast<BMaps16*>(mW1), const_cast<CUtensorMap*>(mHg),
                    const_cast<BMaps*>(mW2), &P};
    int timed = -1;
    DSMOE_TRY(timing_begin(s, &timed));
    DSMOE_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(small_layer_kernel), dim3(G), dim3(SMALL_THREADS),
                                               args, SMEM_BYTES, s));
    DSMOE_TRY(timing_end(s, timed));
    return DSMOE_OK;
}

dsmoe_status launch_layer_umma(const dsmoe_layer_desc& p, const void* x, const void* packed, const float* scores,
                               const uint64_t* mask, const int32_t* k_t, int32_t* counts_out, void* out, char* ws,
                               const WsLayout& L, int32_t* dev_status, cudaStream_t s, bool* done) {
    *done = false;
    (void)k_t;
    if (!umma_supported(p) || p.mode != DSMOE_SELECT_ALL) return DSMOE_OK;
    // Dense forward: gate folded into h, aggregation folded into the down-projection's reduction.
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const __nv_bfloat16* w2t = w1t + (size_t)p.E * p.H * p.d;
    void* hg = ws + L.h;                                        // [T, E*H] bf16
    const CUtensorMap *mA1, *mA2;
    const BMaps *mB1, *mB2;
    DSMOE_TRY(cached_map_2d(&mA1, x, p.T, p.d, BM));
    DSMOE_TRY(cached_bmaps(&mB1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_map_2d(&mA2, hg, p.T, (uint64_t)p.E * p.H, BM));
    DSMOE_TRY(cached_bmaps(&mB2, w2t, p.E, p.d, p.H));
    GemmParams up{};
    up.mode = GEMM_DENSE_UP; up.epi = EPI_GELU; up.E = p.E; up.n_per_expert = p.H; up.k_per_expert = p.d; up.rows = p.T;
    up.gate = scores; up.out = hg; up.ld_out = (long long)p.E * p.H; up.dev_status = dev_status;
    GemmParams down{};
    down.mode = GEMM_DENSE_DOWN; down.epi = EPI_STORE; down.E = p.E; down.n_per_expert = p.d; down.k_per_expert = p.H;
    down.rows = p.T; down.out = out; down.ld_out = p.d; down.out_f32 = p.out_fp32 ? 1 : 0; down.dev_status = dev_status;
    const int mt = ceil_div(p.T, BM);
    const int tiles_up = mt * ceil_div(p.H, BN) * p.E, tiles_down = mt * ceil_div(p.d, BN);
    const int mt2 = ceil_div(p.T, 2 * BM);
    DSMOE_TRY(launch_gemm(*mA1, *mB1, up, tiles_up < sm_count() ? tiles_up : sm_count(), s, true, mt2 * ceil_div(p.H, BN) * p.E));
    DSMOE_TRY(launch_gemm(*mA2, *mB2, down, tiles_down < sm_count() ? tiles_down : sm_count(), s, true, mt2 * ceil_div(p.d, BN)));
    if (counts_out) {
        int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
        int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
        DSMOE_TRY(launch_finalize(p, mask, counts, offsets, reinterpret_cast<int32_t*>(ws + L.chunk_prefix), counts_out, s));
    }
    *done = true;
    return DSMOE_OK;
}

// dS[t,e] = the column tiles' partial sums added in ascending order
__global__ void __launch_bounds__(256) bwd_finish_kernel(const float* __restrict__ part, float* __restrict__ dS, long long n,
                                                         int ntn) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    float v = 0.f;
    for (int j = 0; j < ntn; ++j) v += part[i * ntn + j];
    dS[i] = v;
}

// Gradients of dense training (Eq. 3; Eq. 2 with a mask) on the tensor cores, by recomputation from x:
//   act = GeLU(x.W1[e])            the dense forward's up-projection without the gate     [T, E*H] bf16
//   G   = dO.W2[e]^T               one GEMM over d per expert, W2 read in its natural [H, d] layout
//   dA  = S[t,e] * G,  dS[t,e] = <act[t,e,:], G[t,e,:]>  (= <e_e(x_t), dO_t>)            in that GEMM's epilogue
dsmoe_status launch_dense_backward(const dsmoe_layer_desc& p, const void* x, const void* W2, const void* packed,
                                   const float* scores, const uint64_t* mask, const void* dO, float* dS, void* dA,
                                   void* act, float* dot_part, int32_t* dev_status, cudaStream_t s) {
    if (p.T == 0) return DSMOE_OK;
    if (!umma_supported(p)) return DSMOE_ERR_UNSUPPORTED;
    const __nv_bfloat16* w1t = static_cast<const __nv_bfloat16*>(packed);
    const CUtensorMap *mX, *mdO;
    const BMaps *mB1, *mB2;
    DSMOE_TRY(cached_map_2d(&mX, x, p.T, p.d, BM));
    DSMOE_TRY(cached_bmaps(&mB1, w1t, p.E, p.H, p.d));
    DSMOE_TRY(cached_map_2d(&mdO, dO, p.T, p.d, BM));
    DSMOE_TRY(cached_bmaps_plain(&mB2, W2, p.E, p.H, p.d));
    const long long ld = (long long)p.E * p.H;
    GemmParams up{};
    up.mode = GEMM_DENSE_UP; up.epi = EPI_GELU; up.E = p.E; up.n_per_expert = p.H; up.k_per_expert = p.d; up.rows = p.T;
    up.out = act; up.ld_out = ld; up.dev_status = dev_status;
    GemmParams bw = up;
    bw.epi = EPI_BWD; bw.gate = scores; bw.sel_mask = mask; bw.out = dA; bw.b_plain = 1;
    bw.act = static_cast<const __nv_bfloat16*>(act); bw.dot_part = dot_part;
    const int ntn = ceil_div(p.H, BN);
    const int tiles = ceil_div(p.T, BM) * ntn * p.E;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    const int pair_tiles = ceil_div(p.T, 2 * BM) * ntn * p.E;
    DSMOE_TRY(launch_gemm(*mX, *mB1, up, grid, s, true, pair_tiles));
    DSMOE_TRY(launch_gemm(*mdO, *mB2, bw, grid, s, true, pair_tiles));
    const long long n = (long long)p.T * p.E;
    bwd_finish_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(dot_part, dS, n, ntn);
    DSMOE_CUDA_TRY(cudaGetLastError());
    return DSMOE_OK;
}

}  // namespace dsmoe
