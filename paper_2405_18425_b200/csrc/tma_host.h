// Host-side creation of the tensor maps: 3-D ([units][L][d] bf16, one swizzle span per row) and 4-D (channels-last images).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vig {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeFn encode_fn() {
    static EncodeFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeFn>(p);
    }();
    return fn;
}

// [units][L][d] bf16 tensor, box = [1][rows][row_elems] with row_elems*2 bytes = the swizzle span.
inline bool encode_map(CUtensorMap* map, const void* ptr, long long units, int L, int d, int row_elems, int rows) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)units};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)L * d * 2};
    const cuuint32_t box[3] = {(cuuint32_t)row_elems, (cuuint32_t)rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const int rb = row_elems * 2;
    const CUtensorMapSwizzle sw = rb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                            : (rb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same, through a small cache per host thread: a tensor map is a pure function of the six arguments (it holds the
// address and the shape, nothing of the device's state), and a caller that runs the same buffers again and again - a
// serving loop, a benchmark - would otherwise pay six driver calls of a microsecond or two per forward call.
inline bool make_map(CUtensorMap* map, const void* ptr, long long units, int L, int d, int row_elems, int rows) {
    struct Entry {
        const void* ptr;
        long long units;
        int L, d, row_elems, rows;
        bool valid;
        CUtensorMap map;
    };
    constexpr int kEntries = 64;   // direct-mapped by a hash of the address: six maps per call, ten buffer sets and more fit
    thread_local Entry cache[kEntries] = {};
    const uintptr_t a = reinterpret_cast<uintptr_t>(ptr);
    Entry& e = cache[((a >> 8) ^ (a >> 17) ^ (uintptr_t)(rows * 7 + row_elems)) % kEntries];
    if (e.valid && e.ptr == ptr && e.units == units && e.L == L && e.d == d && e.row_elems == row_elems && e.rows == rows) {
        *map = e.map;
        return true;
    }
    if (!encode_map(map, ptr, units, L, d, row_elems, rows)) return false;
    e.ptr = ptr; e.units = units; e.L = L; e.d = d; e.row_elems = row_elems; e.rows = rows; e.valid = true;
    e.map = *map;
    return true;
}

// [N][Hh][Ww][C] channels-last image tensor of 2- or 4-byte elements, box = [1][box_h][box_w][box_c], no swizzle; reads
// outside the tensor (the zero padding of a convolution, a ragged channel slab) are filled with zeros.  Cached like the
// maps above.
inline bool make_map_nhwc(CUtensorMap* map, const void* ptr, long long N, int Hh, int Ww, int C, int elem, int box_c, int box_w, int box_h) {
    struct Entry {
        const void* ptr;
        long long N;
        int Hh, Ww, C, elem, box_c, box_w, box_h;
        bool valid;
        CUtensorMap map;
    };
    constexpr int kEntries = 16;
    thread_local Entry cache[kEntries] = {};
    const uintptr_t a = reinterpret_cast<uintptr_t>(ptr);
    Entry& e = cache[((a >> 8) ^ (a >> 17)) % kEntries];
    if (e.valid && e.ptr == ptr && e.N == N && e.Hh == Hh && e.Ww == Ww && e.C == C && e.elem == elem && e.box_c == box_c &&
        e.box_w == box_w && e.box_h == box_h) {
        *map = e.map;
        return true;
    }
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)Ww, (cuuint64_t)Hh, (cuuint64_t)N};
    const cuuint64_t strides[3] = {(cuuint64_t)C * elem, (cuuint64_t)Ww * C * elem, (cuuint64_t)Hh * Ww * C * elem};
    const cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (fn(map, elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(ptr), dims, strides, box,
           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.ptr = ptr; e.N = N; e.Hh = Hh; e.Ww = Ww; e.C = C; e.elem = elem; e.box_c = box_c; e.box_w = box_w; e.box_h = box_h; e.valid = true;
    e.map = *map;
    return true;
}

}  // namespace vig
