// Mixture-of-attention-heads layer (Eq. 7-8): the attention step between the two grouped projections.
//
// The layer is the feed-forward layer's pipeline with another middle: router, selection and grouping as there; the
// "up-projection" is the experts' query projection (no activation), the "down-projection" their output projection
// with the router-weighted sum of Eq. 8; in between every grouped row -- one (token, expert) pair, n_head query
// vectors of d_head -- attends to the keys and values of its token's sequence, head j to key/value head j
// (the keys and values are shared by all experts).  This file holds that middle step.
#include <cstdlib>

#include "common.cuh"
#include "tensor_maps.cuh"

namespace dsmoe {

namespace {

constexpr int kMoaWarps = 4;

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// One warp per (grouped row, head).  Pass 1: the lanes share out the visible keys, each key's logit is a full dot
// product of the query (fp32, in shared memory) with the key's row (read in 16-byte pieces); logits go to shared
// memory.  Then max, exponentials and their sum.  Pass 2: the lanes share out the d_head dimensions (lane l owns
// l, l + 32, ...) and walk the keys, so a value row is read by the whole warp at once.  The result replaces the
// query in place (the warp has read all of it before it writes).
template <int DPL>   // d_head / 32
__global__ void __launch_bounds__(32 * kMoaWarps)
moa_attention_kernel(__nv_bfloat16* __restrict__ qa, const int32_t* __restrict__ row_token, const int32_t* __restrict__ offsets,
                     int E, int n_head, int H, int T, const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                     const int32_t* __restrict__ tok_seq, const int32_t* __restrict__ pos, int n_seq, int L, float scale,
                     int* __restrict__ dev_status) {
    constexpr int DH = 32 * DPL;
    extern __shared__ float moa_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* qs = moa_smem + warp * (DH + ((L + 3) & ~3));     // the query, then the logits / probabilities
    float* ws = qs + DH;
    const long long A = offsets[E];
    const long long pair = (long long)blockIdx.x * kMoaWarps + warp;
    if (pair >= A * n_head) return;
    const long long r = pair / n_head;
    const int j = (int)(pair % n_head);
    int t = row_token[r];
    bool bad = t < 0 || t >= T;
    t = min(max(t, 0), T - 1);
    int sq = tok_seq ? tok_seq[t] : 0, last = pos[t];
    bad = bad || sq < 0 || sq >= n_seq || last < 0 || last >= L;
    if (bad) {                                        // report, and stay inside the cache
        if (lane == 0) *dev_status = DSMOE_ERR_INVALID_ARG;
        sq = min(max(sq, 0), n_seq - 1);
        last = min(max(last, 0), L - 1);
    }
    __nv_bfloat16* qrow = qa + r * H + j * DH;
#pragma unroll
    for (int i = 0; i < DPL; ++i) qs[lane + 32 * i] = __bfloat162float(qrow[lane + 32 * i]);
    __syncwarp();
    const __nv_bfloat16* Kh = Kc + ((size_t)(sq * n_head + j) * L) * DH;
    const __nv_bfloat16* Vh = Vc + ((size_t)(sq * n_head + j) * L) * DH;
    float mx = -INFINITY;
    for (int k = lane; k <= last; k += 32) {
        const uint4* kr = reinterpret_cast<const uint4*>(Kh + (size_t)k * DH);
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
            const uint4 u = __ldg(kr + c);
            const float4 q0 = *reinterpret_cast<const float4*>(qs + 8 * c), q1 = *reinterpret_cast<const float4*>(qs + 8 * c + 4);
            dot = fmaf(q0.x, bf16_lo(u.x), dot);
            dot = fmaf(q0.y, bf16_hi(u.x), dot);
            dot = fmaf(q0.z, bf16_lo(u.y), dot);
            dot = fmaf(q0.w, bf16_hi(u.y), dot);
            dot = fmaf(q1.x, bf16_lo(u.z), dot);
            dot = fmaf(q1.y, bf16_hi(u.z), dot);
            dot = fmaf(q1.z, bf16_lo(u.w), dot);
            dot = fmaf(q1.w, bf16_hi(u.w), dot);
        }
        dot *= scale;
        ws[k] = dot;
        mx = fmaxf(mx, dot);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float den = 0.f;
    for (int k = lane; k <= last; k += 32) {
        const float p = expf(ws[k] - mx);
        ws[k] = p;
        den += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    __syncwarp();
    float acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
    for (int k = 0; k <= last; ++k) {
        const float p = ws[k];
        const __nv_bfloat16* vr = Vh + (size_t)k * DH + lane;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] = fmaf(p, __bfloat162float(vr[32 * i]), acc[i]);
    }
    const float inv = 1.f / den;
#pragma unroll
    for (int i = 0; i < DPL; ++i) qrow[lane + 32 * i] = __float2bfloat16_rn(acc[i] * inv);
}

// ---------------------------------------------------------------- the same step on the warp-level tensor-core path
//
// One CTA per (token, head, tile of up to 16 of the token's grouped rows): the rows of a token share its keys and
// values, and 16 rows are exactly the M of an m16n8k16 MMA.  The 8 warps share out the visible keys in blocks of 32:
// a warp copies its block of K and V into (padded, conflict-free) shared memory, forms S = Q.K^T (Q fragments stay
// in registers for the whole kernel), updates the running row maxima and sums, rescales its accumulators and adds
// P.V with P taken straight from S's registers -- the usual streaming-softmax order.  The warps' partial results
// (maximum, sum, accumulator per row) are merged through shared memory at the end, in warp order.  Exponentials are
// the fast ones (ex2.approx of the argument times log2 e): the weights are rounded to bf16 before P.V anyway.
constexpr int kKeyBlock = 32;
#ifndef DSMOE_MOA_MINBLOCKS
#define DSMOE_MOA_MINBLOCKS 6
#endif

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int DH, int kMmaWarps>      // long caches: 8 warps share out the keys; short ones: 2, and several CTAs fit an SM
__global__ void __launch_bounds__(32 * kMmaWarps, kMmaWarps == 2 ? DSMOE_MOA_MINBLOCKS : 1)
moa_attention_mma_kernel(__nv_bfloat16* __restrict__ qa, const int32_t* __restrict__ token_rows, int W, int row_tiles,
                         int tpt, long long amax, int n_head, int H, int T, const __nv_bfloat16* __restrict__ Kc,
                         const __nv_bfloat16* __restrict__ Vc, const int32_t* __restrict__ tok_seq,
                         const int32_t* __restrict__ pos, int n_seq, int L, float scale, long long n_tiles,
                         int* __restrict__ dev_status) {
    constexpr int STRIDE = DH * 2 + 16;                 // bytes per key row in shared memory: 16 of padding
    constexpr int KS = DH / 16, DT = DH / 8, CH = DH / 8;
    extern __shared__ __align__(16) unsigned char moa_mma_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q4 = lane & 3;
    // The tile's 16 rows: with tpt == 1, slots 16 rt .. of token t0; with tpt > 1 (rows per token W <= 8, one row
    // tile), all W slots of the tpt tokens t0, t0 + 1, ...: neighbouring tokens of one sequence see nearly the same
    // keys, so their rows share the copies of K and V.
    // The CTAs are persistent (as many as fit the GPU at once) and walk the tiles: a tile is short, and starting a CTA per
    // tile cost more than the tile's work.
    // With 8 warps (long caches, few tiles) the warps of a CTA share out the KEYS of one tile and merge their partial
    // results at the end; with 2 warps (short caches, many tiles) each warp takes a tile of its OWN, walks all its
    // keys and writes its result straight from registers: no merge, no CTA-wide barrier.
    constexpr bool SPLIT = kMmaWarps > 2;
    constexpr int TW = SPLIT ? 1 : kMmaWarps;           // tiles a CTA works on at a time
    for (long long tile = (long long)blockIdx.x * TW + (SPLIT ? 0 : warp); tile < n_tiles; tile += (long long)gridDim.x * TW) {
    if (SPLIT) __syncthreads();                         // the previous tile's merge has read shared memory
    const int rt = (int)(tile % row_tiles);
    const int j = (int)((tile / row_tiles) % n_head);
    const int t0 = (int)(tile / ((long long)row_tiles * n_head)) * tpt;
    const auto row_token_slot = [&](int i, int& tok, int& slot) {
        if (tpt == 1) {
            tok = t0;
            slot = rt * 16 + i;
        } else {
            tok = t0 + i / W;
            slot = i % W;
            if (i >= tpt * W) tok = T;
        }
    };
    // this thread's two rows of the tile (g and g + 8): grouped row (-1 = none), token, last visible key
    int r0 = -1, r1 = -1, tk0, tk1, sl0, sl1, last0 = 0, last1 = 0;
    row_token_slot(g, tk0, sl0);
    row_token_slot(g + 8, tk1, sl1);
    if (tk0 < T && sl0 < W) r0 = token_rows[(size_t)tk0 * W + sl0];
    if (tk1 < T && sl1 < W) r1 = token_rows[(size_t)tk1 * W + sl1];
    if (r0 >= amax) r0 = -1;
    if (r1 >= amax) r1 = -1;
    if ((SPLIT ? __syncthreads_or(r0 >= 0 || r1 >= 0) : (int)__any_sync(0xffffffffu, r0 >= 0 || r1 >= 0)) == 0) continue;   // no rows in this tile
    bool bad = false;
    if (r0 >= 0) {
        last0 = pos[tk0];
        bad = bad || last0 < 0 || last0 >= L;
        last0 = min(max(last0, 0), L - 1);
    }
    if (r1 >= 0) {
        last1 = pos[tk1];
        bad = bad || last1 < 0 || last1 >= L;
        last1 = min(max(last1, 0), L - 1);
    }
    // the tokens of the tile: one pass over the keys if they all belong to one sequence, else one pass per token
    const int ntok = min(tpt, T - t0);
    int seq_first = tok_seq ? tok_seq[t0] : 0;
    bool same = true;
    for (int u = 1; u < ntok; ++u) same = same && (tok_seq ? tok_seq[t0 + u] : 0) == seq_first;
    const int npass = same ? 1 : ntok;
    // Q fragments (the A operand of S = Q.K^T)
    uint32_t qf[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        const int c = j * DH + ks * 16 + q4 * 2;
        qf[ks][0] = r0 >= 0 ? *reinterpret_cast<const uint32_t*>(qa + (size_t)r0 * H + c) : 0u;
        qf[ks][1] = r1 >= 0 ? *reinterpret_cast<const uint32_t*>(qa + (size_t)r1 * H + c) : 0u;
        qf[ks][2] = r0 >= 0 ? *reinterpret_cast<const uint32_t*>(qa + (size_t)r0 * H + c + 8) : 0u;
        qf[ks][3] = r1 >= 0 ? *reinterpret_cast<const uint32_t*>(qa + (size_t)r1 * H + c + 8) : 0u;
    }
    constexpr int KB = SPLIT ? kKeyBlock / 2 : kKeyBlock;     // keys per block (SPLIT: two buffers of half a block each)
    unsigned char* const Ks0 = moa_mma_smem + (size_t)warp * 2 * kKeyBlock * STRIDE;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    for (int ps = 0; ps < npass; ++ps) {
    // this pass: the sequence whose keys are walked, the rows that take part, the last key any of them sees
    int sq = same ? seq_first : (tok_seq ? tok_seq[t0 + ps] : 0);
    bad = bad || sq < 0 || sq >= n_seq;
    sq = min(max(sq, 0), n_seq - 1);
    const bool act0 = r0 >= 0 && (same || tk0 == t0 + ps), act1 = r1 >= 0 && (same || tk1 == t0 + ps);
    int last = 0;
    for (int u = same ? 0 : ps; u < (same ? ntok : ps + 1); ++u) last = max(last, min(max(pos[t0 + u], 0), L - 1));
    const __nv_bfloat16* Kh = Kc + ((size_t)(sq * n_head + j) * L) * DH;
    const __nv_bfloat16* Vh = Vc + ((size_t)(sq * n_head + j) * L) * DH;
    // Sharing out one tile's keys (SPLIT), a warp walks blocks of KB = 16 keys through two buffers: the copies of its
    // next block are under way while it works on this one (with one buffer of 32 keys and a wait right behind the
    // copies, the decode shape's step took 35 us for 134 MB of keys and values).  A tile per warp: one buffer of 32.
    const int nblocks = last / KB + 1;
    const auto fetch = [&](int b, unsigned char* Kb, unsigned char* Vb) {
        const int key0 = b * KB, nk = min(KB, last + 1 - key0);
#pragma unroll
        for (int i = 0; i < CH * KB / 32; ++i) {        // KB rows x CH 16-byte pieces, a piece per lane and step
            const int idx = lane + 32 * i, row = idx / CH, ch = idx % CH;
            // asynchronous 16-byte copies, all in flight at once; rows past the last visible key are filled with zeros
            const int rr = row < nk ? row : 0;
            const uint32_t nbytes = row < nk ? 16u : 0u;
            const uint32_t kd = (uint32_t)__cvta_generic_to_shared(Kb + row * STRIDE + ch * 16);
            const uint32_t vd = (uint32_t)__cvta_generic_to_shared(Vb + row * STRIDE + ch * 16);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(kd), "l"(Kh + (size_t)(key0 + rr) * DH + ch * 8), "r"(nbytes) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(vd), "l"(Vh + (size_t)(key0 + rr) * DH + ch * 8), "r"(nbytes) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int buf = 0;
    if (SPLIT && warp < nblocks) {
        __syncwarp();
        fetch(warp, Ks0, Ks0 + KB * STRIDE);
    }
    for (int b = SPLIT ? warp : 0; b < nblocks; b += SPLIT ? kMmaWarps : 1) {
        const int key0 = b * KB;
        unsigned char* Ks = Ks0 + buf * 2 * KB * STRIDE;
        unsigned char* Vs = Ks + KB * STRIDE;
        if (SPLIT) {
            __syncwarp();              // the other buffer was last read an iteration ago: every lane is past those reads
            if (b + kMmaWarps < nblocks) {
                unsigned char* Kn = Ks0 + (buf ^ 1) * 2 * KB * STRIDE;
                fetch(b + kMmaWarps, Kn, Kn + KB * STRIDE);
                asm volatile("cp.async.wait_group 1;" ::: "memory");
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
            buf ^= 1;
        } else {
            const int nk = min(KB, last + 1 - key0);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < CH; ++i) {                  // 32 rows x CH 16-byte pieces, a piece per lane and step
                const int idx = lane + 32 * i, row = idx / CH, ch = idx % CH;
                const int rr = row < nk ? row : 0;
                const uint32_t nbytes = row < nk ? 16u : 0u;
                const uint32_t kd = (uint32_t)__cvta_generic_to_shared(Ks + row * STRIDE + ch * 16);
                const uint32_t vd = (uint32_t)__cvta_generic_to_shared(Vs + row * STRIDE + ch * 16);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(kd), "l"(Kh + (size_t)(key0 + rr) * DH + ch * 8), "r"(nbytes) : "memory");
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(vd), "l"(Vh + (size_t)(key0 + rr) * DH + ch * 8), "r"(nbytes) : "memory");
            }
            asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
        }
        __syncwarp();
        float sc[KB / 8][4];
#pragma unroll
        for (int nt = 0; nt < KB / 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int nt = 0; nt < KB / 8; ++nt) {
                const unsigned char* kp = Ks + (nt * 8 + g) * STRIDE + (ks * 16 + q4 * 2) * 2;
                mma_bf16_16816(sc[nt], qf[ks], *reinterpret_cast<const uint32_t*>(kp), *reinterpret_cast<const uint32_t*>(kp + 16));
            }
        }
        // scale, hide the keys past each row's position (and everything from rows not in this pass), new row maxima
        float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < KB / 8; ++nt) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int key = key0 + nt * 8 + q4 * 2 + c;
                sc[nt][c] = (act0 && key <= last0) ? sc[nt][c] * scale : -INFINITY;
                sc[nt][2 + c] = (act1 && key <= last1) ? sc[nt][2 + c] * scale : -INFINITY;
                bm0 = fmaxf(bm0, sc[nt][c]);
                bm1 = fmaxf(bm1, sc[nt][2 + c]);
            }
        }
        bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1));
        bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
        bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1));
        bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
        // a row that has seen no key yet (and sees none here) keeps m = -inf: nothing to rescale, nothing to add
        const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);
        const float c0 = n0 == -INFINITY ? 1.f : __expf(m0 - n0), c1 = n1 == -INFINITY ? 1.f : __expf(m1 - n1);
        m0 = n0;
        m1 = n1;
        l0 *= c0;
        l1 *= c1;
#pragma unroll
        for (int i = 0; i < DT; ++i) {
            o[i][0] *= c0;
            o[i][1] *= c0;
            o[i][2] *= c1;
            o[i][3] *= c1;
        }
        uint32_t pf[KB / 16][4];
#pragma unroll
        for (int nt = 0; nt < KB / 8; ++nt) {
            const float p0 = sc[nt][0] > -INFINITY ? __expf(sc[nt][0] - m0) : 0.f, p1 = sc[nt][1] > -INFINITY ? __expf(sc[nt][1] - m0) : 0.f;
            const float p2 = sc[nt][2] > -INFINITY ? __expf(sc[nt][2] - m1) : 0.f, p3 = sc[nt][3] > -INFINITY ? __expf(sc[nt][3] - m1) : 0.f;
            l0 += p0 + p1;
            l1 += p2 + p3;
            pf[nt / 2][(nt & 1) * 2] = pack_bf16(p0, p1);
            pf[nt / 2][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
#pragma unroll
        for (int kk = 0; kk < KB / 16; ++kk) {
#pragma unroll
            for (int dt = 0; dt < DT; ++dt) {
                uint32_t b0, b1;
                const uint32_t addr = (uint32_t)__cvta_generic_to_shared(Vs + (kk * 16 + (lane & 15)) * STRIDE + dt * 16);
                asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(addr));
                mma_bf16_16816(o[dt], pf[kk], b0, b1);
            }
        }
    }
    }
    if (bad && lane == 0) *dev_status = DSMOE_ERR_INVALID_ARG;             // clamped above: nothing left the cache
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    if (!SPLIT) {
        // the warp has seen every key of its rows: normalise and write (the queries it replaces are in its registers)
        const float i0 = 1.f / l0, i1 = 1.f / l1;
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) {
            const int c = j * DH + dt * 8 + q4 * 2;
            if (r0 >= 0) *reinterpret_cast<uint32_t*>(qa + (size_t)r0 * H + c) = pack_bf16(o[dt][0] * i0, o[dt][1] * i0);
            if (r1 >= 0) *reinterpret_cast<uint32_t*>(qa + (size_t)r1 * H + c) = pack_bf16(o[dt][2] * i1, o[dt][3] * i1);
        }
        continue;
    }
    // ---- merge the warps' partial results: per warp 16 maxima, 16 sums, 16 x DH accumulators
    __syncthreads();
    float* ms = reinterpret_cast<float*>(moa_mma_smem);                 // [warps][16]
    float* ls = ms + kMmaWarps * 16;                                    // [warps][16]
    float* os = ls + kMmaWarps * 16;                                    // [warps][16][DH]
    if (q4 == 0) {
        ms[warp * 16 + g] = m0;
        ms[warp * 16 + g + 8] = m1;
        ls[warp * 16 + g] = l0;
        ls[warp * 16 + g + 8] = l1;
    }
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) {
        float* o0 = os + ((size_t)warp * 16 + g) * DH + dt * 8 + q4 * 2;
        float* o1 = os + ((size_t)warp * 16 + g + 8) * DH + dt * 8 + q4 * 2;
        o0[0] = o[dt][0];
        o0[1] = o[dt][1];
        o1[0] = o[dt][2];
        o1[1] = o[dt][3];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < 16 * DH; idx += 32 * kMmaWarps) {
        const int row = idx / DH, dcol = idx % DH;
        int tok, slot;
        row_token_slot(row, tok, slot);
        if (tok >= T || slot >= W) continue;
        const int r = token_rows[(size_t)tok * W + slot];
        if (r < 0 || r >= amax) continue;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kMmaWarps; ++w) M = fmaxf(M, ms[w * 16 + row]);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int w = 0; w < kMmaWarps; ++w) {
            const float wgt = __expf(ms[w * 16 + row] - M);               // 0 for a warp that saw no key
            num = fmaf(wgt, os[((size_t)w * 16 + row) * DH + dcol], num);
            den = fmaf(wgt, ls[w * 16 + row], den);
        }
        qa[(size_t)r * H + j * DH + dcol] = __float2bfloat16_rn(num / den);
    }
    }
}

template <int DH, int kMmaWarps>
dsmoe_status launch_mma_attention_nw(const dsmoe_layer_desc& p, const MoaCore& c, __nv_bfloat16* q, const int32_t* token_rows,
                                  int32_t* dev_status, cudaStream_t s) {
    constexpr size_t stride = DH * 2 + 16;
    const size_t loop_bytes = (size_t)kMmaWarps * 2 * kKeyBlock * stride;
    const size_t merge_bytes = (size_t)kMmaWarps * (32 + 16 * DH) * 4;
    const size_t smem = loop_bytes > merge_bytes ? loop_bytes : merge_bytes;
    static bool attr[kMaxDeviceSlots] = {};
    int dev = 0;
    DeviceState* st = nullptr;
    DSMOE_TRY(device_state(&st, &dev));
    if (!attr[dev]) {
        DSMOE_CUDA_TRY(cudaFuncSetAttribute(moa_attention_mma_kernel<DH, kMmaWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr[dev] = true;
    }
    const int W = width_of(p), row_tiles = (W + 15) / 16;
    // several tokens per tile where a token has few rows and there are tokens enough to fill the GPU without
    const int tpt = (W <= 8 && (long long)p.T * c.n_head >= 8ll * st->sm_count) ? 16 / W : 1;
    const long long n_tiles = (long long)((p.T + tpt - 1) / tpt) * c.n_head * row_tiles;
    static int per_sm_of[kMaxDeviceSlots] = {};      // CTAs of this kernel that fit an SM, asked once per device
    if (!per_sm_of[dev])
        DSMOE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_of[dev], moa_attention_mma_kernel<DH, kMmaWarps>,
                                                                     32 * kMmaWarps, smem));
    const int per_sm = per_sm_of[dev];
    const long long resident = (long long)st->sm_count * (per_sm > 0 ? per_sm : 1);
    const long long want = kMmaWarps > 2 ? n_tiles : (n_tiles + kMmaWarps - 1) / kMmaWarps;     // 2 warps: a tile per warp
    const long long ctas = want < resident ? want : resident;
    moa_attention_mma_kernel<DH, kMmaWarps><<<(unsigned)ctas, 32 * kMmaWarps, smem, s>>>(
        q, token_rows, W, row_tiles, tpt, (long long)amax_of(p), c.n_head, p.H, p.T, static_cast<const __nv_bfloat16*>(c.Kc),
        static_cast<const __nv_bfloat16*>(c.Vc), c.tok_seq, c.pos, c.n_seq, c.L, c.scale, n_tiles, dev_status);
    return DSMOE_OK;
}

template <int DH>
dsmoe_status launch_mma_attention(const dsmoe_layer_desc& p, const MoaCore& c, __nv_bfloat16* q, const int32_t* token_rows,
                                  int32_t* dev_status, cudaStream_t s) {
    if (c.L <= 512) return launch_mma_attention_nw<DH, 2>(p, c, q, token_rows, dev_status, s);
    return launch_mma_attention_nw<DH, 8>(p, c, q, token_rows, dev_status, s);
}

}  // namespace

bool moa_supported(const dsmoe_layer_desc& p, int n_head, int L) {
    if (!umma_supported(p) || n_head <= 0 || p.H % n_head) return false;
    const int dh = p.H / n_head;
    if (L <= 0 || dh % 32 || dh > 256) return false;
    if (dh == 64 || dh == 96 || dh == 128) return true;                       // tensor-core kernel: any cache length
    return (size_t)(dh + L + 3) * 4 * kMoaWarps <= 200 * 1024;                // plain kernel: a warp's logits sit in shared memory
}

dsmoe_status launch_moa_attention(const dsmoe_layer_desc& p, const MoaCore& c, void* qa, const int32_t* row_token,
                                  const int32_t* token_rows, const int32_t* offsets, int32_t* dev_status, cudaStream_t s) {
    const int dh = p.H / c.n_head;
    // DSMOE_MOA_PLAIN in the environment sends every head width to the plain kernel (a testing aid)
    if (token_rows && (dh == 64 || dh == 96 || dh == 128) && !getenv("DSMOE_MOA_PLAIN")) {
        // head widths of the paper's models: the tensor-core kernel, a CTA per (token, head)
        int timed = -1;
        DSMOE_TRY(timing_begin(s, &timed));
        auto* qb = static_cast<__nv_bfloat16*>(qa);
        if (dh == 64) DSMOE_TRY(launch_mma_attention<64>(p, c, qb, token_rows, dev_status, s));
        else if (dh == 96) DSMOE_TRY(launch_mma_attention<96>(p, c, qb, token_rows, dev_status, s));
        else DSMOE_TRY(launch_mma_attention<128>(p, c, qb, token_rows, dev_status, s));
        DSMOE_CUDA_TRY(cudaGetLastError());
        return timing_end(s, timed);
    }
    int warps = kMoaWarps;
    const size_t per_warp = (size_t)(dh + ((c.L + 3) & ~3)) * 4;
    const size_t smem = per_warp * warps;
    if (smem > 200 * 1024) return DSMOE_ERR_UNSUPPORTED;
    const long long pairs = (long long)amax_of(p) * c.n_head;
    const unsigned grid = (unsigned)((pairs + warps - 1) / warps);
    auto* q = static_cast<__nv_bfloat16*>(qa);
    auto* K = static_cast<const __nv_bfloat16*>(c.Kc);
    auto* V = static_cast<const __nv_bfloat16*>(c.Vc);
    int timed = -1;
    DSMOE_TRY(timing_begin(s, &timed));
#define MOA_LAUNCH(DPL)                                                                                                   \
    do {                                                                                                                  \
        if (smem > 48 * 1024)                                                                                             \
            DSMOE_CUDA_TRY(cudaFuncSetAttribute(moa_attention_kernel<DPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                                (int)smem));                                                              \
        moa_attention_kernel<DPL><<<grid, 32 * kMoaWarps, smem, s>>>(q, row_token, offsets, p.E, c.n_head, p.H, p.T, K, V, \
                                                                     c.tok_seq, c.pos, c.n_seq, c.L, c.scale, dev_status); \
    } while (0)
    switch (dh / 32) {
        case 1: MOA_LAUNCH(1); break;
        case 2: MOA_LAUNCH(2); break;
        case 3: MOA_LAUNCH(3); break;
        case 4: MOA_LAUNCH(4); break;
        case 5: MOA_LAUNCH(5); break;
        case 6: MOA_LAUNCH(6); break;
        case 7: MOA_LAUNCH(7); break;
        case 8: MOA_LAUNCH(8); break;
        default: return DSMOE_ERR_UNSUPPORTED;
    }
#undef MOA_LAUNCH
    DSMOE_CUDA_TRY(cudaGetLastError());
    DSMOE_TRY(timing_end(s, timed));
    return DSMOE_OK;
}

}  // namespace dsmoe
