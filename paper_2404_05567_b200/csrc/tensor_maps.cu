// Tensor maps, per-device facts and the timing ring of the tensor-core launchers (see tensor_maps.cuh).
#include "tensor_maps.cuh"

#include <stdlib.h>

namespace dsmoe {

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
    const cuuint32_t box[2] = {kTileK, box_rows};
    const cuuint32_t es[2] = {1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSMOE_OK : DSMOE_ERR_CUDA;
}

// packed weights of E experts, n output columns, reduction length k: bf16 [E][k / 64][n][64], seen as
// [E][(k / 64) * n][64]; box {64, box_n, 1}, 128-byte swizzle
dsmoe_status make_map_3d(CUtensorMap* m, const void* ptr, uint64_t E, uint64_t n, uint64_t k, uint32_t box_n) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return DSMOE_ERR_CUDA;
    const cuuint64_t dims[3] = {kTileK, (k / kTileK) * n, E};
    const cuuint64_t strides[2] = {kTileK * 2, n * k * 2};
    const cuuint32_t box[3] = {kTileK, box_n, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSMOE_OK : DSMOE_ERR_CUDA;
}

// weights in their natural layout, E matrices [n, k] with k contiguous: bf16 [E][n][k]; box {64 of k, box_n, 1}
dsmoe_status make_map_3d_plain(CUtensorMap* m, const void* ptr, uint64_t E, uint64_t n, uint64_t k, uint32_t box_n) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return DSMOE_ERR_CUDA;
    const cuuint64_t dims[3] = {k, n, E};
    const cuuint64_t strides[2] = {k * 2, n * k * 2};
    const cuuint32_t box[3] = {kTileK, box_n, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSMOE_OK : DSMOE_ERR_CUDA;
}

dsmoe_status make_bmaps16(BMaps16* b, const void* ptr, uint64_t E, uint64_t n, uint64_t k) {
    for (int i = 0; i < 16; ++i) DSMOE_TRY(make_map_3d(&b->m[i], ptr, E, n, k, 16u * (i + 1)));
    return DSMOE_OK;
}

// the five box heights of one packed weight tensor
dsmoe_status make_bmaps(BMaps* b, const void* ptr, uint64_t E, uint64_t n, uint64_t k) {
    for (int lvl = 0; lvl < 5; ++lvl) DSMOE_TRY(make_map_3d(&b->m[lvl], ptr, E, n, k, 16u << lvl));
    return DSMOE_OK;
}

int sm_count() {
    DeviceState* st = nullptr;
    return device_state(&st) == DSMOE_OK ? st->sm_count : 148;   // no device (host-only sizing): the B200's count
}

// Tensor maps depend only on the buffer and the shape, and encoding one is a driver call of a few microseconds
// (a layer call needs up to 23): they are encoded once and found again by (address, shape).  A decode loop or a
// serving loop calls with the same buffers every step.  Not thread-safe, like the rest of the host side.
struct MapKey {
    const void* ptr;
    uint64_t a, b, c;
    int kind;
    bool operator==(const MapKey& o) const { return ptr == o.ptr && a == o.a && b == o.b && c == o.c && kind == o.kind; }
};
template <typename M, int N>
struct MapCache {
    MapKey key[N];
    M map[N];
    int n = 0, next = 0;
    M* find(const MapKey& k) {
        for (int i = 0; i < n; ++i)
            if (key[i] == k) return &map[i];
        return nullptr;
    }
    M* slot(const MapKey& k) {
        const int i = n < N ? n++ : (next++ % N);
        key[i] = k;
        return &map[i];
    }
};
MapCache<CUtensorMap, 256> g_maps2d;
MapCache<BMaps, 128> g_bmaps;
MapCache<BMaps16, 64> g_bmaps16;

dsmoe_status cached_map_2d(const CUtensorMap** out, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    const MapKey k{ptr, rows, cols, box_rows, 0};
    CUtensorMap* m = g_maps2d.find(k);
    if (!m) {
        CUtensorMap tmp;
        DSMOE_TRY(make_map_2d(&tmp, ptr, rows, cols, box_rows));
        m = g_maps2d.slot(k);
        *m = tmp;
    }
    *out = m;
    return DSMOE_OK;
}
dsmoe_status cached_bmaps(const BMaps** out, const void* ptr, uint64_t E, uint64_t n, uint64_t kk) {
    const MapKey k{ptr, E, n, kk, 1};
    BMaps* m = g_bmaps.find(k);
    if (!m) {
        BMaps tmp;
        DSMOE_TRY(make_bmaps(&tmp, ptr, E, n, kk));
        m = g_bmaps.slot(k);
        *m = tmp;
    }
    *out = m;
    return DSMOE_OK;
}
dsmoe_status cached_bmaps_plain(const BMaps** out, const void* ptr, uint64_t E, uint64_t n, uint64_t kk) {
    const MapKey k{ptr, E, n, kk, 3};
    BMaps* m = g_bmaps.find(k);
    if (!m) {
        BMaps tmp;
        for (int lvl = 0; lvl < 5; ++lvl) DSMOE_TRY(make_map_3d_plain(&tmp.m[lvl], ptr, E, n, kk, 16u << lvl));
        m = g_bmaps.slot(k);
        *m = tmp;
    }
    *out = m;
    return DSMOE_OK;
}
dsmoe_status cached_bmaps16(const BMaps16** out, const void* ptr, uint64_t E, uint64_t n, uint64_t kk) {
    const MapKey k{ptr, E, n, kk, 2};
    BMaps16* m = g_bmaps16.find(k);
    if (!m) {
        BMaps16 tmp;
        DSMOE_TRY(make_bmaps16(&tmp, ptr, E, n, kk));
        m = g_bmaps16.slot(k);
        *m = tmp;
    }
    *out = m;
    return DSMOE_OK;
}


// Optional per-launch timing of the tensor-core kernels (a measurement aid for benchmarks): a ring of CUDA event
// pairs; every timed launch takes the next pair until the ring is full.  The events sit on the caller's stream, so a
// benchmark can leave them inside its un-synchronised step loop and read all durations afterwards.
static struct Timing {
    bool on = false;
    int n = 0, cap = 0;
    cudaEvent_t *start = nullptr, *stop = nullptr;
} g_timing;

dsmoe_status timing_begin(cudaStream_t s, int* slot) {
    *slot = -1;
    if (!g_timing.on || g_timing.n >= g_timing.cap) return DSMOE_OK;
    DSMOE_CUDA_TRY(cudaEventRecord(g_timing.start[g_timing.n], s));
    *slot = g_timing.n++;
    return DSMOE_OK;
}

dsmoe_status timing_end(cudaStream_t s, int slot) {
    if (slot >= 0) DSMOE_CUDA_TRY(cudaEventRecord(g_timing.stop[slot], s));
    return DSMOE_OK;
}

dsmoe_status timing_enable(int n_pairs) {
    if (n_pairs > g_timing.cap) {
        cudaEvent_t* a = static_cast<cudaEvent_t*>(realloc(g_timing.start, sizeof(cudaEvent_t) * n_pairs));
        cudaEvent_t* b = static_cast<cudaEvent_t*>(realloc(g_timing.stop, sizeof(cudaEvent_t) * n_pairs));
        if (a) g_timing.start = a;
        if (b) g_timing.stop = b;
        if (!a || !b) return DSMOE_ERR_CUDA;
        for (int i = g_timing.cap; i < n_pairs; ++i) {
            DSMOE_CUDA_TRY(cudaEventCreate(&g_timing.start[i]));
            DSMOE_CUDA_TRY(cudaEventCreate(&g_timing.stop[i]));
            g_timing.cap = i + 1;
        }
    }
    g_timing.on = n_pairs > 0;
    g_timing.n = 0;
    return DSMOE_OK;
}

dsmoe_status timing_read(float* ms, int n_max, int* n) {
    *n = 0;
    for (int i = 0; i < g_timing.n && i < n_max; ++i) {
        DSMOE_CUDA_TRY(cudaEventSynchronize(g_timing.stop[i]));
        DSMOE_CUDA_TRY(cudaEventElapsedTime(&ms[i], g_timing.start[i], g_timing.stop[i]));
        *n = i + 1;
    }
    g_timing.n = 0;
    return DSMOE_OK;
}

}  // namespace dsmoe
