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
// Layer-by-layer entry point (all layers of the range in the same launches, blockIdx.y = layer):
//   per token   the two kernels above with a layer dimension, then one compaction in which every plane
//               reads its own layer's kept list
//   per layer   Eq. 7 as printed: cosines and their per-sequence means, then
//     layer_offsets_kernel  one CTA per layer: which sequences have lost their visual rows at this layer
//                           (the first layer whose mean is under M, and every deeper one), the offsets of
//                           their survivors
//     layer_fill_kernel     the kept positions of every layer in closed form (a dropped sequence keeps the
//                           rows in front of and behind its visual block)
#include <mutex>

#include "common.cuh"
#include "compact.cuh"

namespace sharpv {
namespace {

constexpr int kChunk = 256;             // packed positions per chunk of the flag scan

__host__ __device__ inline size_t ws_flags_bytes(int64_t T) { return ((size_t)T + 255) / 256 * 256; }
__host__ __device__ inline int64_t num_chunks(int64_t T) { return (T + kChunk - 1) / kChunk; }

// element / byte distances between the layers of a layer-by-layer call (all 0 for a single layer)
struct LayerStrides {
    int64_t hidden_bytes, cos, flags, chunks, mean, kept, offsets;
};

constexpr int kRowsPerCta = 4;          // one packed position per warp; small CTAs balance the SMs
constexpr int64_t kInlineBaseChunks = 4096;  // up to this many chunks every chunk CTA adds up the counts in front of it itself
// Up to this many positions no chunk counts are kept at all: a chunk CTA counts the keep flags in front
// of it (one byte a position, 16 to a load, L2-resident), which saves clearing the counters and the
// atomics that fill them.  The cost grows with the square of the positions, hence the limit.
constexpr int64_t kCountFlagsPositions = 65536;
enum BaseSource { kBaseFromCounts = 0, kBaseFromScan = 1, kBaseFromFlags = 2 };

template <int DT>
__global__ void __launch_bounds__(kRowsPerCta * 32)
calibrate_cos_kernel(const char* __restrict__ hidden, int64_t hidden_row_bytes,
                     const char* __restrict__ visual, int64_t visual_row_bytes, int nvec,
                     int num_seqs, const int32_t* __restrict__ seq_offsets,
                     const int32_t* __restrict__ vis_begin, const int32_t* __restrict__ vis_count,
                     const int32_t* __restrict__ vis_offsets, int64_t T, int64_t total_visual, float M,
                     float* __restrict__ out_cos, uint8_t* __restrict__ flags,
                     int32_t* __restrict__ chunk_counts, LayerStrides ls) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t p = (int64_t)blockIdx.x * kRowsPerCta + warp;
    // blockIdx.y is the layer of a layer-by-layer call (0 otherwise): its hidden state and its outputs
    hidden += (int64_t)blockIdx.y * ls.hidden_bytes;
    out_cos += (int64_t)blockIdx.y * ls.cos;
    if (flags) flags += (int64_t)blockIdx.y * ls.flags;
    if (chunk_counts) chunk_counts += (int64_t)blockIdx.y * ls.chunks;
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
    if (lane == 0 && flags) {
        flags[p] = (uint8_t)keep;
        if (keep && chunk_counts) atomicAdd(chunk_counts + p / kChunk, 1);     // integer: order does not matter
    }
}

__global__ void __launch_bounds__(kChunk)
write_kept_kernel(const uint8_t* __restrict__ flags, const int32_t* __restrict__ chunk_counts, int bases_ready,
                  int64_t T, int num_seqs, const int32_t* __restrict__ seq_offsets, int64_t capacity,
                  int32_t* __restrict__ out_kept_pos, int32_t* __restrict__ out_kept_seq_offsets,
                  int32_t* status_word, LayerStrides ls) {
    __shared__ int sm[kChunk / 32 + 1];
    __shared__ int s_base;
    const int c = blockIdx.x;
    flags += (int64_t)blockIdx.y * ls.flags;
    if (chunk_counts) chunk_counts += (int64_t)blockIdx.y * ls.chunks;
    out_kept_pos += (int64_t)blockIdx.y * ls.kept;
    out_kept_seq_offsets += (int64_t)blockIdx.y * ls.offsets;
    cudaGridDependencySynchronize();        // flags and chunk counts come from the kernel in front
    // all global loads of this thread are issued up front: one memory round trip, not three
    const int64_t p = (int64_t)c * kChunk + threadIdx.x;
    const int keep = p < T ? flags[p] : 0;
    // kept positions before this chunk: the counts of the chunks in front, or (many chunks) their
    // exclusive scan, which a one-CTA kernel in front has left in the same array, or (few positions, no
    // counts kept) the keep flags in front, counted here
    int part = 0;
    if (bases_ready == kBaseFromScan) {
        if (threadIdx.x == 0) part = chunk_counts[c];
    } else if (bases_ready == kBaseFromFlags) {
        const uint4* fv = reinterpret_cast<const uint4*>(flags);       // flags are 0 or 1: byte sums by dp4a
        unsigned acc = 0;
        for (int i = threadIdx.x; i < c * (kChunk / 16); i += kChunk) {
            const uint4 w = __ldcg(fv + i);
            acc = __dp4a(w.x, 0x01010101u, acc);
            acc = __dp4a(w.y, 0x01010101u, acc);
            acc = __dp4a(w.z, 0x01010101u, acc);
            acc = __dp4a(w.w, 0x01010101u, acc);
        }
        part = (int)acc;
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
                const int32_t* __restrict__ vis_offsets, int64_t total_visual, float* __restrict__ out_mean,
                LayerStrides ls) {
    __shared__ float part[8];
    const int b = blockIdx.x;
    cosv += (int64_t)blockIdx.y * ls.cos;
    out_mean += (int64_t)blockIdx.y * ls.mean;
    cudaGridDependencySynchronize();
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
    const int bases_ready = total_seq_tokens <= kCountFlagsPositions ? kBaseFromFlags
                            : (int64_t)chunks > kInlineBaseChunks     ? kBaseFromScan
                                                                      : kBaseFromCounts;
    if (bases_ready == kBaseFromFlags) chunk_counts = nullptr;
    // the per-chunk counts are accumulated with atomics and must start at zero
    if (chunk_counts && cudaMemsetAsync(chunk_counts, 0, sizeof(int32_t) * (size_t)chunks, stream) != cudaSuccess)
        return SHARPV_ERR_CUDA;
    {
        auto kern = dtype == SHARPV_F32 ? calibrate_cos_kernel<SHARPV_F32> : calibrate_cos_kernel<SHARPV_BF16>;
        if (launch_dependent(kern, dim3(ctas), dim3(kRowsPerCta * 32), 0, stream, (const char*)hidden, ld_hidden * eb,
                             (const char*)visual, ld_visual * eb, nvec, (int)num_seqs, seq_offsets, vis_begin,
                             vis_count, vis_offsets, total_seq_tokens, total_visual, M, out_cos, flags,
                             chunk_counts, LayerStrides{}) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    if (bases_ready == kBaseFromScan &&
        launch_dependent(exclusive_scan_i32_kernel<false>, dim3(1), dim3(kScanThreads), 0, stream,
                         (const int32_t*)chunk_counts, (int64_t)chunks, 0, chunk_counts, (int32_t*)nullptr,
                         (int32_t*)nullptr, (int64_t)-1, (int32_t*)nullptr) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (launch_dependent(write_kept_kernel, dim3(chunks), dim3(kChunk), 0, stream, (const uint8_t*)flags,
                         (const int32_t*)chunk_counts, bases_ready, total_seq_tokens, num_seqs, seq_offsets, capacity,
                         out_kept_pos, out_kept_seq_offsets, status_word, LayerStrides{}) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (out_mean_cos &&
        launch_dependent(mean_cos_kernel, dim3((unsigned)num_seqs), dim3(256), 0, stream, (const float*)out_cos,
                         vis_count, vis_offsets, total_visual, out_mean_cos, LayerStrides{}) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
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

namespace sharpv {
namespace {

// has sequence b lost its visual rows at layer index li?  (mean under M at li or at a layer in front)
__device__ __forceinline__ bool dropped_at(const float* __restrict__ mean, int num_seqs, int b, int li, float M,
                                           int vis_count_b) {
    if (vis_count_b <= 0) return false;
    for (int i = 0; i <= li; ++i)
        if (mean[(int64_t)i * num_seqs + b] < M) return true;      // Eq. 7: discard iff cos(V_l, V) < M
    return false;
}

// One CTA per layer index: survivors of every sequence at that layer and their exclusive scan.
__global__ void __launch_bounds__(256)
layer_offsets_kernel(const float* __restrict__ mean, int num_seqs, int n_layers, int layer_begin, float M,
                     const int32_t* __restrict__ seq_offsets, const int32_t* __restrict__ vis_count,
                     int64_t capacity, int32_t* __restrict__ out_kept_seq_offsets,
                     int32_t* __restrict__ out_first_discard, int32_t* status_word) {
    __shared__ int sm[256 / 32 + 1];
    const int li = blockIdx.x;
    cudaGridDependencySynchronize();        // the means come from the kernel in front
    int32_t* offsets = out_kept_seq_offsets + (int64_t)li * (num_seqs + 1);
    int carry = 0;
    for (int b0 = 0; b0 < num_seqs; b0 += 256) {
        const int b = b0 + threadIdx.x;
        int cnt = 0;
        if (b < num_seqs) {
            const int vc = vis_count[b];
            cnt = seq_offsets[b + 1] - seq_offsets[b] - (dropped_at(mean, num_seqs, b, li, M, vc) ? vc : 0);
            if (li == 0 && out_first_discard) {
                int first = n_layers;
                for (int i = n_layers - 1; i >= 0; --i)
                    if (vc > 0 && mean[(int64_t)i * num_seqs + b] < M) first = i;
                out_first_discard[b] = layer_begin + first;
            }
        }
        int total;
        const int pre = block_exclusive_scan<256>(cnt, sm, total);
        if (b < num_seqs) offsets[b] = carry + pre;
        carry += total;
    }
    if (threadIdx.x == 0) {
        offsets[num_seqs] = carry;
        if ((int64_t)carry > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    }
}

// Kept positions of every layer: position p of sequence b keeps its place among the survivors, minus
// the visual block if that is gone and p lies behind it.
__global__ void __launch_bounds__(256)
layer_fill_kernel(const float* __restrict__ mean, int num_seqs, float M, const int32_t* __restrict__ seq_offsets,
                  const int32_t* __restrict__ vis_begin, const int32_t* __restrict__ vis_count, int64_t T,
                  int64_t capacity, const int32_t* __restrict__ kept_seq_offsets, int32_t* __restrict__ out_kept_pos) {
    const int li = blockIdx.y;
    const int64_t p = (int64_t)blockIdx.x * 256 + threadIdx.x;
    cudaGridDependencySynchronize();
    if (p >= T) return;
    const int b = upper_segment(seq_offsets, num_seqs, (int)p);
    const int local = (int)p - __ldg(seq_offsets + b);
    const int vb = __ldg(vis_begin + b), vc = __ldg(vis_count + b);
    int rank = local;
    if (dropped_at(mean, num_seqs, b, li, M, vc)) {
        if (local >= vb && local < vb + vc) return;         // a visual row of a sequence that has lost them
        if (local >= vb + vc) rank -= vc;
    }
    const int64_t j = (int64_t)__ldg(kept_seq_offsets + (int64_t)li * (num_seqs + 1) + b) + rank;
    if (j < capacity) out_kept_pos[(int64_t)li * capacity + j] = (int32_t)p;
}

}  // namespace
}  // namespace sharpv

extern "C" size_t sharpv_kv_prune_layers_workspace_bytes(int64_t total_seq_tokens, int32_t num_seqs,
                                                         int32_t num_layers) {
    if (num_layers < 1) num_layers = 1;
    const size_t one = sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens, num_seqs);
    return one * (size_t)num_layers + align_up((size_t)num_layers * (size_t)(num_seqs > 0 ? num_seqs : 1) * 4, 256);
}

// Stage two layer by layer (Section 3.2.3): per token, every layer is calibrated on its own hidden state
// and its planes are compacted with its own kept list; per layer, Eq. 7 as printed.
extern "C" sharpv_status sharpv_kv_prune_layers(
    const void* hidden, int64_t stride_hidden_layer, int64_t ld_hidden, const void* visual, int64_t ld_visual,
    sharpv_dtype dtype, int32_t d, int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets, int64_t total_seq_tokens, int64_t total_visual,
    float M, sharpv_prune_mode mode, float* out_cos, float* out_mean_cos, int32_t* out_first_discard,
    int32_t* out_kept_pos, int32_t* out_kept_seq_offsets, int64_t capacity, const void* kv_src,
    const sharpv_kv_layout* src_layout, void* kv_dst, const sharpv_kv_layout* dst_layout, int32_t layer_begin,
    int32_t layer_end, void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (!src_layout || !dst_layout || layer_begin < 0 || layer_begin > layer_end ||
        layer_end > src_layout->num_layers || stride_hidden_layer < 0 || num_seqs < 1 || capacity < 0 || d < 1 ||
        total_seq_tokens < 0 || total_visual < 0 || ld_hidden < d || ld_visual < d)
        return SHARPV_ERR_INVALID_ARG;
    if ((int)mode < 0 || (int)mode > 1) return SHARPV_ERR_INVALID_ARG;
    if (mode == SHARPV_PRUNE_PER_TOKEN && out_first_discard) return SHARPV_ERR_INVALID_ARG;    // a per-layer output
    const int64_t eb = elem_bytes(dtype);
    if ((stride_hidden_layer * eb) % 16) return SHARPV_ERR_UNSUPPORTED;
    const int n_layers = layer_end - layer_begin;
    if (n_layers == 0) return SHARPV_OK;
    if (!seq_offsets || !vis_begin || !vis_count || !vis_offsets || !out_kept_seq_offsets)
        return SHARPV_ERR_INVALID_ARG;
    if (total_seq_tokens >= (int64_t)1 << 31 || total_visual >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    if (((int64_t)d * eb) % 16 || (ld_hidden * eb) % 16 || (ld_visual * eb) % 16) return SHARPV_ERR_UNSUPPORTED;
    if (workspace_bytes < sharpv_kv_prune_layers_workspace_bytes(total_seq_tokens, num_seqs, n_layers))
        return SHARPV_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (total_seq_tokens == 0) {
        if (cudaMemsetAsync(out_kept_seq_offsets, 0, sizeof(int32_t) * (size_t)n_layers * (num_seqs + 1), stream) !=
            cudaSuccess)
            return SHARPV_ERR_CUDA;
        return SHARPV_OK;
    }
    if (!hidden || !workspace || (capacity > 0 && !out_kept_pos)) return SHARPV_ERR_INVALID_ARG;
    if (total_visual > 0 && (!visual || !out_cos)) return SHARPV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(visual) || !aligned16(workspace)) return SHARPV_ERR_UNSUPPORTED;

    // workspace: per layer (flags | chunk counts), then the means when the caller does not want them
    const size_t one = sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens, num_seqs);
    const unsigned chunks = (unsigned)num_chunks(total_seq_tokens);
    uint8_t* flags = (uint8_t*)workspace;
    int32_t* chunk_counts = (int32_t*)((char*)workspace + ws_flags_bytes(total_seq_tokens));
    float* mean = out_mean_cos ? out_mean_cos : (float*)((char*)workspace + one * (size_t)n_layers);
    LayerStrides ls;
    ls.hidden_bytes = stride_hidden_layer * eb;
    ls.cos = total_visual;
    ls.flags = (int64_t)one;
    ls.chunks = (int64_t)(one / 4);
    ls.mean = num_seqs;
    ls.kept = capacity;
    ls.offsets = num_seqs + 1;
    const bool per_token = mode == SHARPV_PRUNE_PER_TOKEN;
    if (per_token && (int64_t)chunks > kInlineBaseChunks) {
        // more chunks than a chunk CTA adds up by itself: one layer at a time, each with its scan kernel
        for (int32_t l = layer_begin; l < layer_end; ++l) {
            const int64_t i = l - layer_begin;
            int32_t* kp = out_kept_pos ? out_kept_pos + i * capacity : nullptr;
            int32_t* kso = out_kept_seq_offsets + i * (num_seqs + 1);
            sharpv_status st = calibrate_impl(
                (const char*)hidden + i * stride_hidden_layer * eb, ld_hidden, visual, ld_visual, dtype, d, num_seqs,
                seq_offsets, vis_begin, vis_count, vis_offsets, total_seq_tokens, total_visual, M,
                out_cos ? out_cos + i * total_visual : nullptr, out_mean_cos ? out_mean_cos + i * num_seqs : nullptr,
                kp, kso, capacity, workspace, one, status_word, cuda_stream);
            if (st != SHARPV_OK) return st;
            st = sharpv_kv_compact(kv_src, src_layout, kv_dst, dst_layout, l, l + 1, kp, kso, num_seqs, capacity,
                                   status_word, cuda_stream);
            if (st != SHARPV_OK) return st;
        }
        return SHARPV_OK;
    }

    const unsigned ctas = (unsigned)((total_seq_tokens + kRowsPerCta - 1) / kRowsPerCta);
    const int nvec = (int)(d * eb / 16);
    if (n_layers > 65535) return SHARPV_ERR_UNSUPPORTED;
    const bool count_flags = total_seq_tokens <= kCountFlagsPositions;
    if (count_flags) chunk_counts = nullptr;
    if (per_token && !count_flags) {
        // every layer's chunk counters start at zero (they sit `one` bytes apart: clear the whole range)
        if (cudaMemsetAsync(workspace, 0, one * (size_t)n_layers, stream) != cudaSuccess) return SHARPV_ERR_CUDA;
    }
    {
        auto kern = dtype == SHARPV_F32 ? calibrate_cos_kernel<SHARPV_F32> : calibrate_cos_kernel<SHARPV_BF16>;
        if (launch_dependent(kern, dim3(ctas, (unsigned)n_layers), dim3(kRowsPerCta * 32), 0, stream,
                             (const char*)hidden, ld_hidden * eb, (const char*)visual, ld_visual * eb, nvec,
                             (int)num_seqs, seq_offsets, vis_begin, vis_count, vis_offsets, total_seq_tokens,
                             total_visual, M, out_cos, per_token ? flags : (uint8_t*)nullptr,
                             per_token ? chunk_counts : (int32_t*)nullptr, ls) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    if (per_token) {
        if (launch_dependent(write_kept_kernel, dim3(chunks, (unsigned)n_layers), dim3(kChunk), 0, stream,
                             (const uint8_t*)flags, (const int32_t*)chunk_counts,
                             (int)(count_flags ? kBaseFromFlags : kBaseFromCounts), total_seq_tokens, num_seqs,
                             seq_offsets, capacity, out_kept_pos, out_kept_seq_offsets, status_word, ls) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    if (!per_token || out_mean_cos) {
        if (launch_dependent(mean_cos_kernel, dim3((unsigned)num_seqs, (unsigned)n_layers), dim3(256), 0, stream,
                             (const float*)out_cos, vis_count, vis_offsets, total_visual, mean, ls) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    if (!per_token) {
        if (launch_dependent(layer_offsets_kernel, dim3((unsigned)n_layers), dim3(256), 0, stream, (const float*)mean,
                             (int)num_seqs, n_layers, (int)layer_begin, M, seq_offsets, vis_count, capacity,
                             out_kept_seq_offsets, out_first_discard, status_word) != cudaSuccess ||
            launch_dependent(layer_fill_kernel, dim3((unsigned)((total_seq_tokens + 255) / 256), (unsigned)n_layers),
                             dim3(256), 0, stream, (const float*)mean, (int)num_seqs, M, seq_offsets, vis_begin,
                             vis_count, total_seq_tokens, capacity, (const int32_t*)out_kept_seq_offsets,
                             out_kept_pos) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    if (!kv_src && !kv_dst) return SHARPV_OK;   // decisions only
    return kv_compact_launch(kv_src, src_layout, kv_dst, dst_layout, layer_begin, layer_end, out_kept_pos,
                             out_kept_seq_offsets + num_seqs, capacity, num_seqs + 1, capacity, status_word, stream);
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
