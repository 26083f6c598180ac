// Microbenchmark: how fast can one SM stream memory with TMA tile copies, as a function of the copy's size and of
// the number of copies it keeps in flight?  Every CTA (one per SM) walks its own part of a 2 GiB buffer with copies of
// `rows` x 128 bytes, `depth` of them outstanding.  The answer shapes the decode kernels: what counts is the NUMBER
// of copies under way (a handful per SM), so each copy has to be large.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>

#include "umma.cuh"

using namespace dsmoe;

__global__ void __launch_bounds__(256, 1) stream_kernel(const __grid_constant__ CUtensorMap tm, int rows, int depth,
                                                       int copies_per_cta, int evict_first, long long rows_total,
                                                       long long span_rows, unsigned long long* gave_up) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ uint64_t full_all[64];
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 64; ++i) ptx::mbar_init(ptx::smem_u32(&full_all[i]), 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    // `issuers` warps (blockDim.x / 32) each run the same single-thread loop on their own slots and their own share
    // of the CTA's copies: does the copy rate depend on how many threads issue?
    if (threadIdx.x & 31) return;
    const int issuer = threadIdx.x >> 5, issuers = blockDim.x >> 5;
    uint64_t* full = full_all + issuer * depth;
    copies_per_cta /= issuers;
    const uint64_t pol = ptx::policy_evict_first();
    const uint32_t bytes = (uint32_t)rows * 128u;
    const uint32_t base = base0 + (uint32_t)issuer * depth * bytes;
    // span_rows > 0: the CTA keeps re-reading its own span_rows rows (small enough for all spans to stay in L2)
    const long long r0 = span_rows > 0 ? (long long)blockIdx.x * span_rows + (long long)issuer * (span_rows / issuers)
                                       : ((long long)blockIdx.x * issuers + issuer) * copies_per_cta * rows;
    auto issue = [&](int n, int slot) {
        const uint32_t bar = ptx::smem_u32(&full[slot]);
        ptx::mbar_expect_tx(bar, bytes);
        const int row = span_rows > 0 ? (int)(r0 + ((long long)n * rows) % (span_rows / issuers)) : (int)((r0 + (long long)n * rows) % rows_total);
        if (evict_first) ptx::tma_load_3d_hint(base + slot * bytes, &tm, bar, 0, row, 0, pol);
        else ptx::tma_load_3d(base + slot * bytes, &tm, bar, 0, row, 0);
    };
    int issued = 0, done = 0, s = 0;
    uint32_t ph = 0;
    for (; issued < depth && issued < copies_per_cta; ++issued) issue(issued, issued);
    while (done < copies_per_cta) {
        if (!ptx::mbar_wait(ptx::smem_u32(&full[s]), ph, &abort_flag)) break;     // bounded wait
        ++done;
        if (issued < copies_per_cta) issue(issued++, s);
        if (++s == depth) {
            s = 0;
            ph ^= 1u;
        }
    }
    if (abort_flag) *gave_up = 1;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int main() {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return 1;
    EncodeTiledFn encode = (EncodeTiledFn)p;
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    const long long bytes = 2ll << 30, rows_total = bytes / 128;
    void* buf = nullptr;
    unsigned long long* gave_up = nullptr;
    if (cudaMalloc(&buf, bytes) != cudaSuccess || cudaMalloc(&gave_up, 8) != cudaSuccess) return 1;
    cudaMemset(buf, 1, bytes);
    cudaMemset(gave_up, 0, 8);
    cudaFuncSetAttribute(stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 170 * 1024);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int rows_list[] = {16, 32, 64, 128, 256};
    for (int from_l2 = 0; from_l2 < 2; ++from_l2)
    for (int rows : rows_list) {
        if (rows == 16)
            printf("%d SMs; source: %s; GB/s over all SMs, best of 3 launches of 4 MiB per SM (L2 evict-first hint: without / with)\n", sms,
                   from_l2 ? "L2 (every SM re-reads its own 512 KiB)" : "HBM (2 GiB walked once)");
        const long long span_rows = from_l2 ? (512 * 1024) / 128 : 0;
        CUtensorMap tm;
        const cuuint64_t dims[3] = {64, (cuuint64_t)rows_total, 1}, strides[2] = {128, (cuuint64_t)bytes};
        const cuuint32_t box[3] = {64, (cuuint32_t)rows, 1}, es[3] = {1, 1, 1};
        if (encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, buf, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return 1;
        for (int issuers = 1; issuers <= 4; issuers *= 2)
        for (int depth = 1; depth <= 32; depth *= 2) {
            if ((long long)issuers * depth * rows * 128 > 160 * 1024 || issuers * depth > 64) continue;
            if (issuers > 1 && depth != 2 && depth != 4) continue;
            float gbs[2];
            for (int hint = 0; hint < 2; ++hint) {
                if (from_l2 && hint) {       // evict-first makes no sense for data that is meant to stay
                    gbs[1] = gbs[0];
                    continue;
                }
                const long long per_cta = 4ll << 20;
                const int copies = (int)(per_cta / (rows * 128));
                float best = 1e9f;
                for (int rep = 0; rep < 3; ++rep) {
                    cudaEventRecord(e0);
                    stream_kernel<<<sms, 32 * issuers, 170 * 1024>>>(tm, rows, depth, copies, hint, rows_total, span_rows, gave_up);
                    cudaEventRecord(e1);
                    cudaEventSynchronize(e1);
                    float ms;
                    cudaEventElapsedTime(&ms, e0, e1);
                    best = ms < best ? ms : best;
                }
                gbs[hint] = (float)((double)sms * per_cta / best / 1e6);
            }
            printf("copy %6d B  x %2d in flight x %d issuing warps = %7d B per SM : %7.1f / %7.1f GB/s   (%.2f copies per us and SM)\n",
                   rows * 128, depth, issuers, issuers * depth * rows * 128, gbs[0], gbs[1], gbs[1] * 1e3 / sms / (rows * 128));
        }
    }
    unsigned long long h = 0;
    cudaMemcpy(&h, gave_up, 8, cudaMemcpyDeviceToHost);
    printf("bounded waits expired: %llu; last CUDA error: %s\n", h, cudaGetErrorString(cudaGetLastError()));
    return 0;
}
