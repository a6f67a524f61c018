// Shared device helpers of the SharpV CUDA library: 128-bit loads, exact widening of
// bf16 / fp32 storage to fp32, warp and block reductions, argument checks.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sharpv.h"

namespace sharpv {

constexpr int kWarp = 32;
constexpr float kNormEps = 1e-12f;      // v^ = v / max(||v||, kNormEps)

// ---------------------------------------------------------------------------------------
// host-side argument checks
// ---------------------------------------------------------------------------------------
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int elem_bytes(sharpv_dtype dt) { return dt == SHARPV_F32 ? 4 : (dt == SHARPV_BF16 ? 2 : 1); }
inline bool dtype_ok(sharpv_dtype dt) { return dt == SHARPV_F32 || dt == SHARPV_BF16; }
inline bool copy_dtype_ok(sharpv_dtype dt) { return dtype_ok(dt) || dt == SHARPV_U8; }    // bit copies only
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Byte range [lo, hi) that the first `rows` token rows of every plane of the layers
// [layer_begin, layer_end) can touch (strides are non-negative, so the range starts at the first
// layer's K block and ends behind the last row of the last layer's last V head).
inline void kv_extent(const void* base, const sharpv_kv_layout* L, int layer_begin, int layer_end, int64_t rows,
                      uintptr_t& lo, uintptr_t& hi) {
    const int64_t eb = elem_bytes(L->dtype);
    lo = reinterpret_cast<uintptr_t>(base) + (uintptr_t)(layer_begin * L->stride_layer * eb);
    hi = reinterpret_cast<uintptr_t>(base) +
         (uintptr_t)(((layer_end - 1) * L->stride_layer + L->stride_kv + (L->num_kv_heads - 1) * L->stride_head +
                      (rows - 1) * L->stride_token + L->head_dim) * eb);
}

// Rows a plane of this layout can hold if the cache is laid out without gaps: the smallest stride above
// the token stride, in token strides.  Only the debug build's range checks use it.
inline int64_t kv_row_limit(const sharpv_kv_layout* L) {
    int64_t best = INT64_MAX;
    const int64_t strides[3] = {L->stride_layer, L->stride_kv, L->stride_head};
    for (int i = 0; i < 3; ++i)
        if (strides[i] > L->stride_token && strides[i] / L->stride_token < best) best = strides[i] / L->stride_token;
    return best == INT64_MAX ? ((int64_t)1 << 31) : best;
}

// true when the first `rows` rows of the planes of [layer_begin, layer_end) of two caches share bytes
inline bool kv_ranges_overlap(const void* a, const sharpv_kv_layout* la, const void* b, const sharpv_kv_layout* lb,
                              int layer_begin, int layer_end, int64_t rows) {
    if (layer_end <= layer_begin || rows <= 0) return false;
    uintptr_t a_lo, a_hi, b_lo, b_hi;
    kv_extent(a, la, layer_begin, layer_end, rows, a_lo, a_hi);
    kv_extent(b, lb, layer_begin, layer_end, rows, b_lo, b_hi);
    return a_lo < b_hi && b_lo < a_hi;
}

inline sharpv_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? SHARPV_OK : SHARPV_ERR_CUDA;
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while the kernel in
// front of it on the stream drains, and must call cudaGridDependencySynchronize() before it reads
// anything that kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------------------
// 16-byte vectors of the storage type and their exact fp32 widening
// ---------------------------------------------------------------------------------------
template <int DT> struct Elem;

template <> struct Elem<SHARPV_F32> {
    static constexpr int kPerVec = 4;
    static constexpr int kBytes = 4;
    __device__ __forceinline__ static void widen(const uint4& v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
};

template <> struct Elem<SHARPV_BF16> {
    static constexpr int kPerVec = 8;
    static constexpr int kBytes = 2;
    // a bf16 is the upper half of an fp32: element 2j is the low half-word, 2j+1 the high one
    __device__ __forceinline__ static void widen(const uint4& v, float (&x)[8]) {
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

// streaming 128-bit load: read-only path, do not keep the line in L1
__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// 128-bit load that may stay in L1/L2 (small tables, frame means)
__device__ __forceinline__ uint4 ld_cached(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}

__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---------------------------------------------------------------------------------------
// reductions (fixed order: results do not depend on scheduling)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Exclusive scan of one int per thread over a block of NT threads (NT a multiple of 32,
// at most 1024).  `total` receives the block sum.  `smem` holds NT/32 + 1 ints.
template <int NT>
__device__ __forceinline__ int block_exclusive_scan(int v, int* smem, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = lane < NT / 32 ? smem[lane] : 0;
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        if (lane < NT / 32) smem[lane] = winc - w;      // exclusive warp offsets
        if (lane == 31) smem[NT / 32] = winc;           // block total
    }
    __syncthreads();
    int res = smem[warp] + inc - v;
    total = smem[NT / 32];
    __syncthreads();                                     // smem may be reused by the caller
    return res;
}

// largest b with offsets[b] <= x, for an ascending table offsets[0..n] (offsets[0] <= x < offsets[n])
__device__ __forceinline__ int upper_segment(const int32_t* __restrict__ offsets, int n, int x) {
    int lo = 0, hi = n;          // answer in [lo, hi)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(offsets + mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// same search on a table any address space may hold (shared memory copies of an offset table)
__device__ __forceinline__ int upper_segment_any(const int32_t* offsets, int n, int x) {
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (offsets[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Monotone map fp32 -> uint32: larger score, larger key.  Adding +0 turns -0 into +0.
__device__ __forceinline__ uint32_t order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ void report(int32_t* status_word, int code) {
    if (status_word) atomicMax(status_word, code);
}

// Range check of an index right before it is used for a gather or a scatter.  In a library built with
// -DSHARPV_DEBUG_BOUNDS a violation is recorded in the status word and the caller skips the access; in
// the release build the check compiles away.
#ifdef SHARPV_DEBUG_BOUNDS
__device__ __forceinline__ bool index_ok(bool in_range, int32_t* status_word) {
    if (!in_range) report(status_word, SHARPV_ERR_BOUNDS);
    return in_range;
}
#else
__device__ __forceinline__ bool index_ok(bool, int32_t*) { return true; }
#endif

// Exclusive prefix sums of n ints by one CTA of 1024 threads: thread i adds up a contiguous share,
// one block scan, then every thread writes the prefixes of its share.  out[i] = sum of val(in[j]),
// j < i, with val = min(max(in[j], 0), clamp_hi) when CLAMP; out == in is allowed.  If out_total is
// not null it receives the grand total (as do *total_copy, if not null, and the capacity check).
constexpr int kScanThreads = 1024;
template <bool CLAMP>
__global__ void __launch_bounds__(kScanThreads)
exclusive_scan_i32_kernel(const int32_t* in, int64_t n, int clamp_hi, int32_t* out, int32_t* out_total,
                          int32_t* total_copy, int64_t capacity, int32_t* status_word) {
    __shared__ int sm[kScanThreads / 32 + 1];
    cudaGridDependencySynchronize();
    const int64_t per = (n + kScanThreads - 1) / kScanThreads;
    const int64_t lo = min(n, (int64_t)threadIdx.x * per), hi = min(n, lo + per);
    int sum = 0;
    for (int64_t i = lo; i < hi; ++i) {
        const int v = in[i];
        sum += CLAMP ? min(max(v, 0), clamp_hi) : v;
    }
    int total;
    int run = block_exclusive_scan<kScanThreads>(sum, sm, total);
    for (int64_t i = lo; i < hi; ++i) {
        const int v = in[i];
        out[i] = run;
        run += CLAMP ? min(max(v, 0), clamp_hi) : v;
    }
    if (threadIdx.x == 0) {
        if (out_total) *out_total = total;
        if (total_copy) *total_copy = total;
        if (capacity >= 0 && (int64_t)total > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    }
}

}  // namespace sharpv
