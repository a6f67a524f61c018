// Stage two (a): self-calibrated degradation test (Section 3.2.3, Eq. 7) per visual token,
// followed by the compaction of the keep flags into ascending kept positions.
//
// Kernels:
//   calibrate_cos_kernel  one warp per packed position: cos(hidden row, visual row), keep flag,
//                         and an integer count of survivors per chunk of 256 positions
//   write_kept_kernel     (dependent launch) chunk base = sum of earlier chunk counts (beyond 4096 chunks a
//                         one-CTA scan kernel in front turns the counts into bases), local scan,
//                         ascending kept positions, per-sequence offsets, capacity check
//   mean_cos_kernel       (optional) fixed-order mean of the cosines of each sequence
#include <mutex>

#include "common.cuh"

namespace sharpv {
namespace {

constexpr int kChunk = 256;             // packed positions per chunk of the flag scan

__host__ __device__ inline size_t ws_flags_bytes(int64_t T) { return ((size_t)T + 255) / 256 * 256; }
__host__ __device__ inline int64_t num_chunks(int64_t T) { return (T + kChunk - 1) / kChunk; }

constexpr int kRowsPerCta = 4;          // one packed position per warp; small CTAs balance the SMs
constexpr int64_t kInlineBaseChunks = 4096;  // up to this many chunks every chunk CTA adds up the counts in front of it itself

template <int DT>
__global__ void __launch_bounds__(kRowsPerCta * 32)
calibrate_cos_kernel(const char* __restrict__ hidden, int64_t hidden_row_bytes,
                     const char* __restrict__ visual, int64_t visual_row_bytes, int nvec,
                     int num_seqs, const int32_t* __restrict__ seq_offsets,
                     const int32_t* __restrict__ vis_begin, const int32_t* __restrict__ vis_count,
                     const int32_t* __restrict__ vis_offsets, int64_t T, int64_t total_visual, float M,
                     float* __restrict__ out_cos, uint8_t* __restrict__ flags,
                     int32_t* __restrict__ chunk_counts) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t p = (int64_t)blockIdx.x * kRowsPerCta + warp;
    cudaGridDependencySynchronize();        // hidden states and counters come from earlier work on the stream
    if (p >= T) return;
    const int b = upper_segment(seq_offsets, num_seqs, (int)p);
    const int64_t local = p - __ldg(seq_offsets + b) - __ldg(vis_begin + b);
    int keep = 1;
    if (local >= 0 && local < __ldg(vis_count + b)) {
        const int64_t vrow = (int64_t)__ldg(vis_offsets + b) + local;
        if (vrow < total_visual) {
            const char* ph = hidden + p * hidden_row_bytes;
            const char* pv = visual + vrow * visual_row_bytes;
            float shh = 0.f, svv = 0.f, shv = 0.f;
            int v = lane;
            for (; v + 96 < nvec; v += 128) {           // 8 independent 128-bit loads in flight
                uint4 rh[4], rv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    rh[u] = ld_stream(ph + (int64_t)(v + 32 * u) * 16);
                    rv[u] = ld_stream(pv + (int64_t)(v + 32 * u) * 16);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float h[P], x[P];
                    E::widen(rh[u], h);
                    E::widen(rv[u], x);
#pragma unroll
                    for (int j = 0; j < P; ++j) {
                        shh = fmaf(h[j], h[j], shh);
                        svv = fmaf(x[j], x[j], svv);
                        shv = fmaf(h[j], x[j], shv);
                    }
                }
            }
            for (; v < nvec; v += 32) {
                float h[P], x[P];
                E::widen(ld_stream(ph + (int64_t)v * 16), h);
                E::widen(ld_stream(pv + (int64_t)v * 16), x);
#pragma unroll
                for (int j = 0; j < P; ++j) {
                    shh = fmaf(h[j], h[j], shh);
                    svv = fmaf(x[j], x[j], svv);
                    shv = fmaf(h[j], x[j], shv);
                }
            }
            shh = warp_sum(shh); svv = warp_sum(svv); shv = warp_sum(shv);
            const float nh = fmaxf(sqrtf(shh), kNormEps), nv = fmaxf(sqrtf(svv), kNormEps);
            const float c = shv / (nh * nv);
            keep = c < M ? 0 : 1;                       // Eq. 7: discard iff cos < M
            if (lane == 0) out_cos[vrow] = c;
        }
    }
    if (lane == 0) {
        flags[p] = (uint8_t)keep;
        if (keep) atomicAdd(chunk_counts + p / kChunk, 1);     // integer: order does not matter
    }
}

__global__ void __launch_bounds__(kChunk)
write_kept_kernel(const uint8_t* __restrict__ flags, const int32_t* __restrict__ chunk_counts, int bases_ready,
                  int64_t T, int num_seqs, const int32_t* __restrict__ seq_offsets, int64_t capacity,
                  int32_t* __restrict__ out_kept_pos, int32_t* __restrict__ out_kept_seq_offsets,
                  int32_t* status_word) {
    __shared__ int sm[kChunk / 32 + 1];
    __shared__ int s_base;
    const int c = blockIdx.x;
    cudaGridDependencySynchronize();        // flags and chunk counts come from the kernel in front
    // all global loads of this thread are issued up front: one memory round trip, not three
    const int64_t p = (int64_t)c * kChunk + threadIdx.x;
    const int keep = p < T ? flags[p] : 0;
    // kept positions before this chunk: the counts of the chunks in front, or (many chunks) their
    // exclusive scan, which a one-CTA kernel in front has left in the same array
    int part = 0;
    if (bases_ready) {
        if (threadIdx.x == 0) part = chunk_counts[c];
    } else {
        for (int i = threadIdx.x; i < c; i += kChunk) part += chunk_counts[i];
    }
    int seq_first = -1, seq_last = -1;      // sequences that start at p: [seq_first, seq_last]
    if (p < T) {
        int b = upper_segment(seq_offsets, num_seqs, (int)p);
        if (__ldg(seq_offsets + b) == (int)p) {
            seq_last = b;
            while (b > 0 && __ldg(seq_offsets + b - 1) == (int)p) --b;
            seq_first = b;
        }
    }
    // kept positions before this chunk: fixed-order sum of the earlier chunk counts
    int total_before;
    block_exclusive_scan<kChunk>(part, sm, total_before);
    if (threadIdx.x == 0) s_base = total_before;
    __syncthreads();
    const int base = s_base;

    int chunk_total;
    const int rank = block_exclusive_scan<kChunk>(keep, sm, chunk_total);
    const int64_t j = (int64_t)base + rank;
    if (keep && j < capacity) out_kept_pos[j] = (int32_t)p;
    for (int b = seq_first; b >= 0 && b <= seq_last; ++b) out_kept_seq_offsets[b] = (int32_t)j;

    if (c == gridDim.x - 1 && threadIdx.x == 0) {
        const int64_t total = (int64_t)base + chunk_total;
        // trailing empty sequences and the end marker
        for (int b = num_seqs; b >= 0 && __ldg(seq_offsets + b) >= T; --b) out_kept_seq_offsets[b] = (int32_t)total;
        if (total > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    }
}

__global__ void __launch_bounds__(256)
mean_cos_kernel(const float* __restrict__ cosv, const int32_t* __restrict__ vis_count,
                const int32_t* __restrict__ vis_offsets, int64_t total_visual, float* __restrict__ out_mean) {
    __shared__ float part[8];
    const int b = blockIdx.x;
    const int n = vis_count[b];
    const int64_t o = vis_offsets[b];
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += 256)
        if (o + i < total_visual) s += cosv[o + i];
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += part[i];
        out_mean[b] = n > 0 ? tot / (float)n : 0.f;
    }
}

}  // namespace
}  // namespace sharpv

using namespace sharpv;

extern "C" size_t sharpv_kv_calibrate_prune_workspace_bytes(int64_t total_seq_tokens, int32_t num_seqs) {
    (void)num_seqs;
    if (total_seq_tokens <= 0) return 256;
    return ws_flags_bytes(total_seq_tokens) + align_up((size_t)num_chunks(total_seq_tokens) * 4, 256);
}

static sharpv_status calibrate_impl(
    const void* hidden, int64_t ld_hidden, const void* visual, int64_t ld_visual, sharpv_dtype dtype,
    int32_t d, int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets, int64_t total_seq_tokens, int64_t total_visual,
    float M, float* out_cos, float* out_mean_cos, int32_t* out_kept_pos, int32_t* out_kept_seq_offsets,
    int64_t capacity, void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (num_seqs < 1 || d < 1 || total_seq_tokens < 0 || total_visual < 0 || capacity < 0 || ld_hidden < d ||
        ld_visual < d)
        return SHARPV_ERR_INVALID_ARG;
    if (!seq_offsets || !vis_begin || !vis_count || !vis_offsets || !out_kept_seq_offsets)
        return SHARPV_ERR_INVALID_ARG;
    if (total_seq_tokens >= (int64_t)1 << 31 || total_visual >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    const int eb = elem_bytes(dtype);
    if (((int64_t)d * eb) % 16 || (ld_hidden * eb) % 16 || (ld_visual * eb) % 16) return SHARPV_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (total_seq_tokens == 0) {
        if (cudaMemsetAsync(out_kept_seq_offsets, 0, sizeof(int32_t) * (size_t)(num_seqs + 1), stream) != cudaSuccess)
            return SHARPV_ERR_CUDA;
        if (out_mean_cos &&
            cudaMemsetAsync(out_mean_cos, 0, sizeof(float) * (size_t)num_seqs, stream) != cudaSuccess)
            return SHARPV_ERR_CUDA;
        return SHARPV_OK;
    }
    if (!hidden || !workspace || (capacity > 0 && !out_kept_pos)) return SHARPV_ERR_INVALID_ARG;
    if (total_visual > 0 && (!visual || !out_cos)) return SHARPV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(visual) || !aligned16(workspace)) return SHARPV_ERR_UNSUPPORTED;
    if (workspace_bytes < sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens, num_seqs))
        return SHARPV_ERR_WORKSPACE;

    uint8_t* flags = (uint8_t*)workspace;
    int32_t* chunk_counts = (int32_t*)((char*)workspace + ws_flags_bytes(total_seq_tokens));
    const unsigned chunks = (unsigned)num_chunks(total_seq_tokens);
    const unsigned ctas = (unsigned)((total_seq_tokens + kRowsPerCta - 1) / kRowsPerCta);
    const int nvec = d * eb / 16;
    // the per-chunk counts are accumulated with atomics and must start at zero
    if (cudaMemsetAsync(chunk_counts, 0, sizeof(int32_t) * (size_t)chunks, stream) != cudaSuccess)
        return SHARPV_ERR_CUDA;
    {
        auto kern = dtype == SHARPV_F32 ? calibrate_cos_kernel<SHARPV_F32> : calibrate_cos_kernel<SHARPV_BF16>;
        if (launch_dependent(kern, dim3(ctas), dim3(kRowsPerCta * 32), 0, stream, (const char*)hidden, ld_hidden * eb,
                             (const char*)visual, ld_visual * eb, nvec, (int)num_seqs, seq_offsets, vis_begin,
                             vis_count, vis_offsets, total_seq_tokens, total_visual, M, out_cos, flags,
                             chunk_counts) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    const int bases_ready = (int64_t)chunks > kInlineBaseChunks;
    if (bases_ready &&
        launch_dependent(exclusive_scan_i32_kernel<false>, dim3(1), dim3(kScanThreads), 0, stream,
                         (const int32_t*)chunk_counts, (int64_t)chunks, 0, chunk_counts, (int32_t*)nullptr,
                         (int32_t*)nullptr, (int64_t)-1, (int32_t*)nullptr) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (launch_dependent(write_kept_kernel, dim3(chunks), dim3(kChunk), 0, stream, (const uint8_t*)flags,
                         (const int32_t*)chunk_counts, bases_ready, total_seq_tokens, num_seqs, seq_offsets, capacity,
                         out_kept_pos, out_kept_seq_offsets, status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (out_mean_cos)
        mean_cos_kernel<<<num_seqs, 256, 0, stream>>>(out_cos, vis_count, vis_offsets, total_visual, out_mean_cos);
    return launch_status();
}

extern "C" sharpv_status sharpv_kv_calibrate_prune(
    const void* hidden, int64_t ld_hidden, const void* visual, int64_t ld_visual, sharpv_dtype dtype,
    int32_t d, int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets, int64_t total_seq_tokens, int64_t total_visual,
    float M, float* out_cos, float* out_mean_cos, int32_t* out_kept_pos, int32_t* out_kept_seq_offsets,
    int64_t capacity, void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    return calibrate_impl(hidden, ld_hidden, visual, ld_visual, dtype, d, num_seqs, seq_offsets, vis_begin,
                          vis_count, vis_offsets, total_seq_tokens, total_visual, M, out_cos, out_mean_cos,
                          out_kept_pos, out_kept_seq_offsets, capacity, workspace, workspace_bytes, status_word,
                          cuda_stream);
}

// Stage two layer by layer: every layer in the range is calibrated on its own hidden state and only
// its own K/V planes are compacted with its own kept list (Section 3.2.3 read per layer).
extern "C" sharpv_status sharpv_kv_prune_layers(
    const void* hidden, int64_t stride_hidden_layer, int64_t ld_hidden, const void* visual, int64_t ld_visual,
    sharpv_dtype dtype, int32_t d, int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets, int64_t total_seq_tokens, int64_t total_visual,
    float M, float* out_cos, float* out_mean_cos, int32_t* out_kept_pos, int32_t* out_kept_seq_offsets,
    int64_t capacity, const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst,
    const sharpv_kv_layout* dst_layout, int32_t layer_begin, int32_t layer_end, void* workspace,
    size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (!src_layout || !dst_layout || layer_begin < 0 || layer_begin > layer_end ||
        layer_end > src_layout->num_layers || stride_hidden_layer < 0 || num_seqs < 1 || capacity < 0)
        return SHARPV_ERR_INVALID_ARG;
    if ((stride_hidden_layer * elem_bytes(dtype)) % 16) return SHARPV_ERR_UNSUPPORTED;
    const int64_t eb = elem_bytes(dtype);
    for (int32_t l = layer_begin; l < layer_end; ++l) {
        const int64_t i = l - layer_begin;
        int32_t* kept_pos = out_kept_pos ? out_kept_pos + i * capacity : nullptr;
        int32_t* kept_seq_offsets = out_kept_seq_offsets ? out_kept_seq_offsets + i * (num_seqs + 1) : nullptr;
        sharpv_status st = calibrate_impl(
            hidden ? (const char*)hidden + i * stride_hidden_layer * eb : nullptr, ld_hidden, visual, ld_visual, dtype,
            d, num_seqs, seq_offsets, vis_begin, vis_count, vis_offsets, total_seq_tokens, total_visual, M,
            out_cos ? out_cos + i * total_visual : nullptr, out_mean_cos ? out_mean_cos + i * num_seqs : nullptr,
            kept_pos, kept_seq_offsets, capacity, workspace, workspace_bytes, status_word, cuda_stream);
        if (st != SHARPV_OK) return st;
        st = sharpv_kv_compact(kv_src, src_layout, kv_dst, dst_layout, l, l + 1, kept_pos, kept_seq_offsets, num_seqs,
                               capacity, status_word, cuda_stream);
        if (st != SHARPV_OK) return st;
    }
    return SHARPV_OK;
}

// ---------------------------------------------------------------------------------------
// Allocation-free variant: the scratch lives in a file-scope device array
// ---------------------------------------------------------------------------------------
namespace {

constexpr int64_t kNoAllocMaxTokens = SHARPV_NOALLOC_MAX_SEQ_TOKENS;
constexpr size_t kNoAllocScratchBytes =
    ((size_t)kNoAllocMaxTokens + 255) / 256 * 256 +                                   // keep flags
    (((size_t)(kNoAllocMaxTokens + kChunk - 1) / kChunk) * 4 + 255) / 256 * 256;      // per-chunk counts

// Held by every GPU that loads this library until the process exits (about 260 KB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};     // device address of g_noalloc_scratch, per device

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can
// use: the device address has to be asked for, once per device, with that device current.
sharpv_status noalloc_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SHARPV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return SHARPV_OK;
}

}  // namespace

extern "C" sharpv_status sharpv_kv_calibrate_prune_noalloc(
    const void* hidden, int64_t ld_hidden, const void* visual, int64_t ld_visual, sharpv_dtype dtype,
    int32_t d, int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets, int64_t total_seq_tokens, int64_t total_visual,
    float M, float* out_cos, float* out_mean_cos, int32_t* out_kept_pos, int32_t* out_kept_seq_offsets,
    int64_t capacity, int32_t* status_word, void* cuda_stream) {
    if (total_seq_tokens > kNoAllocMaxTokens) return SHARPV_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    const sharpv_status st = noalloc_scratch(&scratch);
    if (st != SHARPV_OK) return st;
    // Every flag below total_seq_tokens is rewritten before it is read and the chunk counts are
    // cleared on the stream at the start of each call, so the previous call leaves nothing behind.
    return calibrate_impl(hidden, ld_hidden, visual, ld_visual, dtype, d, num_seqs, seq_offsets, vis_begin,
                          vis_count, vis_offsets, total_seq_tokens, total_visual, M, out_cos, out_mean_cos,
                          out_kept_pos, out_kept_seq_offsets, capacity, scratch, kNoAllocScratchBytes,
                          status_word, cuda_stream);
}
