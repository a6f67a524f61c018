// Stage one (b): per-frame top-k of the importance scores with a stable tie-break, the
// exclusive scan of the budgets, and the gather of the kept token rows
// (Section 3.1, first paragraph; Section 3.1.3, last paragraph).
//
// Kernels:
//   count_above_kernel   (threshold variant only) per-frame count of I > K
//   select_frame_kernel  one CTA per frame: its offset (sum of the budgets in front of it; beyond 4096
//                        frames a one-CTA scan kernel in front computes all offsets), then in
//                        shared memory either a rank count over composite (key, index) keys (frames
//                        of up to 1024 tokens) or a 4-pass byte radix select of the k-th largest key
//                        with an index-ordered scan for the tie-break; ascending indices out
//   gather_rows_kernel   one warp per kept row, 128-bit copies; launched as a dependent of the
//                        selection so that its start-up overlaps it
#include "common.cuh"

namespace sharpv {
namespace {

constexpr int kSelectThreads = 256;
constexpr int kMaxTokensPerFrame = 8192;
constexpr int kRankMaxTokens = 1024;     // frames up to this size are selected by counting ranks
constexpr int kInlineOffsetFrames = 4096; // up to this many frames every frame CTA adds up the budgets in front of it itself

__global__ void __launch_bounds__(kSelectThreads)
count_above_kernel(const float* __restrict__ importance, float K, int f, int32_t* __restrict__ counts) {
    __shared__ int part[kSelectThreads / 32];
    const int t = blockIdx.x;
    int c = 0;
    for (int i = threadIdx.x; i < f; i += kSelectThreads) c += importance[(int64_t)t * f + i] > K;
    c = warp_sum_int(c);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int i = 0; i < kSelectThreads / 32; ++i) tot += part[i];
        counts[t] = tot;
    }
}

// mode 0: top-k with budgets k[t];  mode 1: keep I > K
__global__ void __launch_bounds__(kSelectThreads)
select_frame_kernel(const float* __restrict__ importance, const int32_t* __restrict__ k, int F, int f,
                    int64_t capacity, int mode, float K, int offsets_ready, int32_t* __restrict__ kept_offsets,
                    int32_t* __restrict__ num_kept, int32_t* __restrict__ out_kept_index, int32_t* status_word) {
    extern __shared__ __align__(16) uint32_t keys[];   // [f]
    __shared__ int hist[4][256];                       // one histogram per byte pass, cleared once
    __shared__ int scan_sm[kSelectThreads / 32 + 1];
    __shared__ int off_sm[kSelectThreads / 32];
    __shared__ int s_digit, s_remaining;

    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* imp = importance + (int64_t)t * f;
    cudaGridDependencySynchronize();        // scores and budgets come from earlier work on the stream

    // this frame's offset: the (clamped) budgets of the frames in front of it, added in a fixed order
    // here, or read from the scan a kernel in front has left in kept_offsets (large batches)
    int part = 0;
    if (!offsets_ready)
        for (int i = tid; i < t; i += kSelectThreads) part += min(max(k[i], 0), f);
    const int kt_raw = k[t];
    for (int i = tid; i < f; i += kSelectThreads) keys[i] = mode == 0 ? order_key(imp[i]) : (imp[i] > K ? 1u : 0u);
    for (int i = tid; i < 4 * 256; i += kSelectThreads) (&hist[0][0])[i] = 0;
    part = warp_sum_int(part);
    if (lane == 0) off_sm[warp] = part;
    __syncthreads();
    int before = 0;
    if (offsets_ready) {
        before = kept_offsets[t];
    } else {
#pragma unroll
        for (int i = 0; i < kSelectThreads / 32; ++i) before += off_sm[i];
    }
    const int64_t out_base = before;
    if (tid == 0 && !offsets_ready) {
        kept_offsets[t] = before;
        if (t == F - 1) {
            const int total = before + min(max(kt_raw, 0), f);
            kept_offsets[F] = total;
            if (num_kept) *num_kept = total;
            if ((int64_t)total > capacity) report(status_word, SHARPV_ERR_CAPACITY);
        }
    }

    uint32_t kth = 0;
    int remaining = 0;
    bool keep_all = false;
    if (mode == 0) {
        const int kt = min(max(kt_raw, 0), f);
        if (kt == 0) return;
        keep_all = kt == f;
        if (!keep_all && f <= kRankMaxTokens) {
            // Small frames: a token's rank under (key descending, index ascending) is the number of
            // composite keys (key, ~index) above its own; it is kept iff rank < k.  No histogram,
            // no pass structure: one sweep over shared memory, then one scan for the positions.
            unsigned long long* comp = reinterpret_cast<unsigned long long*>(keys + ((f + 3) & ~3));
            const int fpad = (f + 1) & ~1;
            for (int i = tid; i < fpad; i += kSelectThreads)
                comp[i] = i < f ? (((unsigned long long)keys[i] << 32) | (0xffffffffu - (uint32_t)i)) : 0ull;
            __syncthreads();
            int carry = 0;
            for (int base = 0; base < f; base += kSelectThreads) {
                const int i = base + tid;
                const bool valid = i < f;
                const unsigned long long mine = valid ? comp[i] : ~0ull;
                int rank = 0;
                for (int j = 0; j < fpad; j += 2) {
                    const ulonglong2 c = *reinterpret_cast<const ulonglong2*>(comp + j);
                    rank += (c.x > mine) + (c.y > mine);
                }
                const bool keep = valid && rank < kt;
                int total;
                const int pos = carry + block_exclusive_scan<kSelectThreads>(keep ? 1 : 0, scan_sm, total);
                carry += total;
                if (keep) {
                    const int64_t j = out_base + pos;
                    if (j < capacity) out_kept_index[j] = t * f + i;
                }
            }
            return;
        }
        if (!keep_all) {
            // radix select, most significant byte first: after the four passes `prefix` is the
            // k-th largest key and `remaining` says how many keys equal to it are still owed
            uint32_t prefix = 0, mask = 0;
            remaining = kt;
            int pass = 0;
            for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
                for (int i = tid; i < f; i += kSelectThreads) {
                    const uint32_t key = keys[i];
                    if ((key & mask) == prefix) atomicAdd(&hist[pass][(key >> shift) & 255u], 1);
                }
                __syncthreads();
                if (warp == 0) {
                    const int top = 255 - lane * 8;    // lane 0 owns the 8 largest digits
                    int c[8], sum = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { c[j] = hist[pass][top - j]; sum += c[j]; }
                    int inc = sum;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        int n = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc += n;
                    }
                    int acc = inc - sum;               // candidates with a larger digit than my range
                    if (acc < remaining && remaining <= inc) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (acc < remaining && remaining <= acc + c[j]) {
                                s_digit = top - j;
                                s_remaining = remaining - acc;
                            }
                            acc += c[j];
                        }
                    }
                }
                __syncthreads();
                prefix |= (uint32_t)s_digit << shift;
                mask |= 0xffu << shift;
                remaining = s_remaining;
            }
            kth = prefix;
        }
    }
    // threshold variant: keys are 1 (kept) or 0, kth = 0, remaining = 0: "greater than 0" keeps them

    // index-ordered pass: keys above the k-th are kept; among keys equal to it the first `remaining`
    // in index order are kept.  One scan carries both counts (low half: greater, high half: equal).
    int carry = 0;
    for (int base = 0; base < f; base += kSelectThreads) {
        const int i = base + tid;
        const bool valid = i < f;
        const uint32_t key = valid ? keys[i] : 0u;
        const bool gt = valid && (keep_all || key > kth);
        const bool eq = valid && !keep_all && key == kth && remaining > 0;
        int total;
        const int pre = carry + block_exclusive_scan<kSelectThreads>((gt ? 1 : 0) | (eq ? 1 << 16 : 0), scan_sm, total);
        carry += total;
        const int gt_before = pre & 0xffff, eq_before = pre >> 16;
        if (gt || (eq && eq_before < remaining)) {
            const int64_t j = out_base + gt_before + min(eq_before, remaining);
            if (j < capacity) out_kept_index[j] = t * f + i;
        }
    }
}

// one warp per half row, up to eight 128-bit loads in flight per lane
__global__ void __launch_bounds__(256)
gather_rows_kernel(const char* __restrict__ src, int64_t src_row_bytes, int64_t src_rows, int nvec,
                   const int32_t* __restrict__ index, const int32_t* __restrict__ count_ptr,
                   int64_t capacity, char* __restrict__ dst, int64_t dst_row_bytes, int32_t* status_word) {
    cudaGridDependencySynchronize();        // the index list comes from the kernel in front
    const int lane = threadIdx.x & 31;
    const int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int64_t j = w >> 1;
    if (j >= capacity) return;
    // the count and the index are fetched together (slot j exists even when it holds no index yet)
    const int32_t row_index = __ldg(index + j);
    const int64_t n = min((int64_t)__ldg(count_ptr), capacity);
    if (j >= n) return;
    if (!index_ok(row_index >= 0 && row_index < src_rows, status_word)) return;
    const int half = (nvec + 1) >> 1;
    const int v0 = (int)(w & 1) * half, v1 = min(nvec, v0 + half);
    const char* s = src + (int64_t)row_index * src_row_bytes;
    char* o = dst + j * dst_row_bytes;
    for (int v = v0 + lane; v < v1; v += 256) {
        uint4 r[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (v + 32 * u < v1) r[u] = ld_stream(s + (int64_t)(v + 32 * u) * 16);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (v + 32 * u < v1) st_stream(o + (int64_t)(v + 32 * u) * 16, r[u]);
    }
}

sharpv_status select_impl(int mode, const float* importance, const int32_t* k, float K, int32_t F, int32_t f,
                          const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t d,
                          int32_t* out_kept_index, int32_t* out_kept_offsets, void* out_tokens,
                          int64_t capacity, int32_t* out_num_kept, void* workspace, size_t workspace_bytes,
                          int32_t* status_word, void* cuda_stream) {
    if (F < 0 || f < 1 || capacity < 0) return SHARPV_ERR_INVALID_ARG;
    if (!out_kept_offsets) return SHARPV_ERR_INVALID_ARG;
    if (f > kMaxTokensPerFrame) return SHARPV_ERR_UNSUPPORTED;
    if ((int64_t)F * f >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    if (F > 0 && (!importance || (mode == 0 && !k))) return SHARPV_ERR_INVALID_ARG;
    if (capacity > 0 && !out_kept_index) return SHARPV_ERR_INVALID_ARG;
    int eb = 0;
    if (out_tokens) {
        if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
        if (!tokens || d < 1 || ld_tokens < d) return SHARPV_ERR_INVALID_ARG;
        eb = elem_bytes(dtype);
        if (((int64_t)d * eb) % 16 || (ld_tokens * eb) % 16 || !aligned16(tokens) || !aligned16(out_tokens))
            return SHARPV_ERR_UNSUPPORTED;
    }
    if (workspace_bytes < sharpv_select_tokens_workspace_bytes(F, f)) return SHARPV_ERR_WORKSPACE;
    if (F > 0 && !workspace) return SHARPV_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    const int32_t* budgets = k;
    if (mode == 1 && F > 0) {
        int32_t* counts = (int32_t*)workspace;
        count_above_kernel<<<F, kSelectThreads, 0, stream>>>(importance, K, f, counts);
        if (launch_status() != SHARPV_OK) return SHARPV_ERR_CUDA;
        budgets = counts;
    }
    if (F == 0) {
        if (cudaMemsetAsync(out_kept_offsets, 0, sizeof(int32_t), stream) != cudaSuccess) return SHARPV_ERR_CUDA;
        if (out_num_kept && cudaMemsetAsync(out_num_kept, 0, sizeof(int32_t), stream) != cudaSuccess)
            return SHARPV_ERR_CUDA;
        return SHARPV_OK;
    }
    // keys, plus the 64-bit composite keys of the rank-counting path for small frames
    const size_t sel_smem = (size_t)((f + 3) & ~3) * 4 + (f <= kRankMaxTokens ? (size_t)((f + 1) & ~1) * 8 : 0);
    const int offsets_ready = F > kInlineOffsetFrames;
    if (offsets_ready &&
        launch_dependent(exclusive_scan_i32_kernel<true>, dim3(1), dim3(kScanThreads), 0, stream, budgets, (int64_t)F,
                         (int)f, out_kept_offsets, out_kept_offsets + F, out_num_kept, capacity, status_word) !=
            cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (launch_dependent(select_frame_kernel, dim3((unsigned)F), dim3(kSelectThreads), sel_smem, stream,
                         importance, budgets, (int)F, (int)f, capacity, mode, K, offsets_ready, out_kept_offsets,
                         out_num_kept, out_kept_index, status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (out_tokens && capacity > 0) {
        const int64_t rows = capacity < (int64_t)F * f ? capacity : (int64_t)F * f;
        const int nvec = d * eb / 16;
        if (launch_dependent(gather_rows_kernel, dim3((unsigned)((2 * rows + 7) / 8)), dim3(256), 0, stream,
                             (const char*)tokens, ld_tokens * eb, (int64_t)F * f, nvec, (const int32_t*)out_kept_index,
                             (const int32_t*)(out_kept_offsets + F), capacity, (char*)out_tokens,
                             (int64_t)d * eb, status_word) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    return SHARPV_OK;
}

}  // namespace
}  // namespace sharpv

using namespace sharpv;

extern "C" size_t sharpv_select_tokens_workspace_bytes(int32_t total_frames, int32_t f) {
    (void)f;
    return align_up((size_t)(total_frames > 0 ? total_frames : 1) * 4, 256);
}

extern "C" sharpv_status sharpv_select_tokens(
    const float* importance, const int32_t* k, int32_t total_frames, int32_t f, const void* tokens,
    sharpv_dtype dtype, int64_t ld_tokens, int32_t d, int32_t* out_kept_index, int32_t* out_kept_offsets,
    void* out_tokens, int64_t capacity, int32_t* out_num_kept, void* workspace, size_t workspace_bytes,
    int32_t* status_word, void* cuda_stream) {
    return select_impl(0, importance, k, 0.f, total_frames, f, tokens, dtype, ld_tokens, d, out_kept_index,
                       out_kept_offsets, out_tokens, capacity, out_num_kept, workspace, workspace_bytes,
                       status_word, cuda_stream);
}

extern "C" sharpv_status sharpv_select_tokens_threshold(
    const float* importance, float K, int32_t total_frames, int32_t f, const void* tokens,
    sharpv_dtype dtype, int64_t ld_tokens, int32_t d, int32_t* out_kept_index, int32_t* out_kept_offsets,
    void* out_tokens, int64_t capacity, int32_t* out_num_kept, void* workspace, size_t workspace_bytes,
    int32_t* status_word, void* cuda_stream) {
    return select_impl(1, importance, nullptr, K, total_frames, f, tokens, dtype, ld_tokens, d, out_kept_index,
                       out_kept_offsets, out_tokens, capacity, out_num_kept, workspace, workspace_bytes,
                       status_word, cuda_stream);
}
