// Stage two (b): K/V compaction (Section 3.2.3).  For every (layer, K|V, head) plane the rows
// of the kept positions are copied, in order, to a dense prefix of the destination plane.
// One index list serves all planes.
//
// Out of place: persistent CTAs walk the (plane, tile) list with 128-bit loads and stores through
// registers.  In place (kv_dst == kv_src): one CTA per plane, front to back.
// Bulk async copies (one cp.async.bulk per kept 256-byte row into a shared-memory tile, one bulk
// store per dense tile) were measured and lost: the copy engine's per-request cost caps 256-byte
// rows near 2.2 TB/s of reads, against 2.7 TB/s for this kernel at the same kept share.
#include "common.cuh"

namespace sharpv {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kCompactUnroll = 4;         // 16-byte vectors in flight per thread
constexpr int kCompactCtasPerSm = 5;      // resident CTAs per SM at 47 registers

struct PlaneGeom {
    int64_t src_layer, src_kv, src_head, src_token;     // bytes
    int64_t dst_layer, dst_kv, dst_head, dst_token;     // bytes
    int num_kv_heads, layer_begin, row_vecs;            // row_vecs = 16-byte vectors per row
};

// Persistent CTAs walk the (plane, tile) list; a tile is kTileRows destination rows.  Each thread
// moves kUnroll 16-byte vectors per tile, all loads issued before the first store.
template <int kUnroll>
__global__ void __launch_bounds__(kCompactThreads)
kv_compact_kernel(const char* __restrict__ src, char* __restrict__ dst, PlaneGeom g, int planes,
                  const int32_t* __restrict__ kept_pos, const int32_t* __restrict__ n_kept_ptr,
                  int64_t capacity, int32_t* status_word) {
    cudaGridDependencySynchronize();        // the index list and the cache come from earlier work on the stream
    const int64_t n_all = __ldg(n_kept_ptr);
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_all > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    const int64_t n = min(n_all, capacity);
    if (n <= 0) return;
    const int tile_rows = kCompactThreads * kUnroll / g.row_vecs;      // >= 1, checked by the host
    const int64_t tiles_per_plane = (n + tile_rows - 1) / tile_rows;
    const int64_t total_tiles = tiles_per_plane * planes;
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int plane = (int)(tile / tiles_per_plane);
        const int64_t row0 = (tile - plane * tiles_per_plane) * tile_rows;
        const int l = g.layer_begin + plane / (2 * g.num_kv_heads);
        const int kv = (plane / g.num_kv_heads) & 1;
        const int h = plane % g.num_kv_heads;
        const char* s = src + l * g.src_layer + kv * g.src_kv + h * g.src_head;
        char* o = dst + l * g.dst_layer + kv * g.dst_kv + h * g.dst_head;
        const int rows = (int)min((int64_t)tile_rows, n - row0);
        const int total = rows * g.row_vecs;
        uint4 r[kUnroll];
        int64_t off[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int q = threadIdx.x + u * kCompactThreads;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                const int64_t j = row0 + rr;
                r[u] = ld_stream(s + (int64_t)__ldg(kept_pos + j) * g.src_token + (int64_t)vv * 16);
                off[u] = j * g.dst_token + (int64_t)vv * 16;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int q = threadIdx.x + u * kCompactThreads;
            if (q < total) st_stream(o + off[u], r[u]);
        }
    }
}

// In-place compaction (kv_dst == kv_src).  Row j of the result comes from row kept_pos[j] >= j, so a
// tile of destination rows [j0, j0 + R) only reads rows at or behind j0: rows read by later tiles are
// never overwritten by earlier ones, but a tile may overwrite rows that an earlier tile still has to
// read.  One CTA therefore walks a plane front to back: the loads of tile k+1 are issued, a block
// barrier orders every thread's loads of tile k before anybody's stores of tile k, then tile k is
// stored while tile k+1 is in flight.
constexpr int kInplaceThreads = 512;
constexpr int kInplaceUnroll = 4;

__global__ void __launch_bounds__(kInplaceThreads)
kv_compact_inplace_kernel(char* __restrict__ kv, PlaneGeom g, const int32_t* __restrict__ kept_pos,
                          const int32_t* __restrict__ n_kept_ptr, int64_t capacity, int32_t* status_word) {
    cudaGridDependencySynchronize();
    const int64_t n_all = __ldg(n_kept_ptr);
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_all > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    const int64_t n = min(n_all, capacity);
    if (n <= 0) return;
    const int plane = blockIdx.x;
    const int l = g.layer_begin + plane / (2 * g.num_kv_heads);
    const int kvi = (plane / g.num_kv_heads) & 1;
    const int h = plane % g.num_kv_heads;
    char* base = kv + l * g.src_layer + kvi * g.src_kv + h * g.src_head;
    const int tile_rows = kInplaceThreads * kInplaceUnroll / g.row_vecs;
    const int64_t tiles = (n + tile_rows - 1) / tile_rows;

    uint4 cur[kInplaceUnroll], nxt[kInplaceUnroll];
    auto load_tile = [&](int64_t k, uint4 (&r)[kInplaceUnroll]) {
        const int64_t row0 = k * tile_rows;
        const int total = (int)min((int64_t)tile_rows, n - row0) * g.row_vecs;
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) {
            const int q = threadIdx.x + u * kInplaceThreads;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                r[u] = *reinterpret_cast<const uint4*>(base + (int64_t)__ldg(kept_pos + row0 + rr) * g.src_token +
                                                       (int64_t)vv * 16);
            }
        }
    };
    load_tile(0, cur);
    for (int64_t k = 0; k < tiles; ++k) {
        if (k + 1 < tiles) load_tile(k + 1, nxt);
        __syncthreads();                        // every load of tile k happened before any store of tile k
        const int64_t row0 = k * tile_rows;
        const int total = (int)min((int64_t)tile_rows, n - row0) * g.row_vecs;
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) {
            const int q = threadIdx.x + u * kInplaceThreads;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                *reinterpret_cast<uint4*>(base + (row0 + rr) * g.src_token + (int64_t)vv * 16) = cur[u];
            }
        }
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) cur[u] = nxt[u];
    }
}

bool layout_ok(const sharpv_kv_layout* L) {
    return L && L->num_layers >= 1 && L->num_kv_heads >= 1 && L->head_dim >= 1 && copy_dtype_ok(L->dtype) &&
           L->stride_layer >= 0 && L->stride_kv >= 0 && L->stride_head >= 0 && L->stride_token >= L->head_dim;
}

bool layout_aligned(const sharpv_kv_layout* L) {
    const int64_t eb = elem_bytes(L->dtype);
    return (L->head_dim * eb) % 16 == 0 && (L->stride_layer * eb) % 16 == 0 && (L->stride_kv * eb) % 16 == 0 &&
           (L->stride_head * eb) % 16 == 0 && (L->stride_token * eb) % 16 == 0;
}

}  // namespace
}  // namespace sharpv

using namespace sharpv;

extern "C" sharpv_status sharpv_kv_compact(
    const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst, const sharpv_kv_layout* dst_layout,
    int32_t layer_begin, int32_t layer_end, const int32_t* kept_pos, const int32_t* kept_seq_offsets,
    int32_t num_seqs, int64_t capacity, int32_t* status_word, void* cuda_stream) {
    if (!layout_ok(src_layout) || !layout_ok(dst_layout)) {
        if (src_layout && dst_layout && (!copy_dtype_ok(src_layout->dtype) || !copy_dtype_ok(dst_layout->dtype)))
            return SHARPV_ERR_UNSUPPORTED;
        return SHARPV_ERR_INVALID_ARG;
    }
    if (src_layout->dtype != dst_layout->dtype || src_layout->head_dim != dst_layout->head_dim ||
        src_layout->num_kv_heads != dst_layout->num_kv_heads || src_layout->num_layers != dst_layout->num_layers)
        return SHARPV_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > src_layout->num_layers || layer_begin > layer_end || num_seqs < 1 ||
        capacity < 0)
        return SHARPV_ERR_INVALID_ARG;
    if (!kv_src || !kv_dst || !kept_seq_offsets) return SHARPV_ERR_INVALID_ARG;
    const bool in_place = kv_src == kv_dst;
    if (in_place && (src_layout->stride_layer != dst_layout->stride_layer ||
                     src_layout->stride_kv != dst_layout->stride_kv ||
                     src_layout->stride_head != dst_layout->stride_head ||
                     src_layout->stride_token != dst_layout->stride_token))
        return SHARPV_ERR_INVALID_ARG;
    if (capacity > 0 && !kept_pos) return SHARPV_ERR_INVALID_ARG;
    if (!layout_aligned(src_layout) || !layout_aligned(dst_layout) || !aligned16(kv_src) || !aligned16(kv_dst))
        return SHARPV_ERR_UNSUPPORTED;
    if (capacity >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    const int planes = (layer_end - layer_begin) * 2 * src_layout->num_kv_heads;
    if (planes == 0 || capacity == 0) return SHARPV_OK;
    if (planes > 65535) return SHARPV_ERR_UNSUPPORTED;
    if (!in_place) {
        // a destination that shares bytes with the source without being the source itself would be
        // overwritten while other CTAs still read it
        if (kv_ranges_overlap(kv_src, src_layout, kv_dst, dst_layout, layer_begin, layer_end, capacity))
            return SHARPV_ERR_INVALID_ARG;
    }

    const int64_t eb = elem_bytes(src_layout->dtype);
    PlaneGeom g;
    g.src_layer = src_layout->stride_layer * eb; g.src_kv = src_layout->stride_kv * eb;
    g.src_head = src_layout->stride_head * eb;   g.src_token = src_layout->stride_token * eb;
    g.dst_layer = dst_layout->stride_layer * eb; g.dst_kv = dst_layout->stride_kv * eb;
    g.dst_head = dst_layout->stride_head * eb;   g.dst_token = dst_layout->stride_token * eb;
    g.num_kv_heads = src_layout->num_kv_heads;
    g.layer_begin = layer_begin;
    g.row_vecs = (int)(src_layout->head_dim * eb / 16);
    if (g.row_vecs > kCompactThreads * kCompactUnroll) return SHARPV_ERR_UNSUPPORTED;    // rows over 16 KB
    if (in_place) {
        if (launch_dependent(kv_compact_inplace_kernel, dim3((unsigned)planes), dim3(kInplaceThreads), 0,
                             (cudaStream_t)cuda_stream, (char*)kv_dst, g, kept_pos, kept_seq_offsets + num_seqs,
                             capacity, status_word) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
        return SHARPV_OK;
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    const int tile_rows = kCompactThreads * kCompactUnroll / g.row_vecs;
    const int64_t max_tiles = (capacity + tile_rows - 1) / tile_rows * planes;
    const int64_t want = (int64_t)sms * kCompactCtasPerSm;
    const unsigned grid = (unsigned)(max_tiles < want ? max_tiles : want);
    if (launch_dependent(kv_compact_kernel<kCompactUnroll>, dim3(grid), dim3(kCompactThreads), 0,
                         (cudaStream_t)cuda_stream, (const char*)kv_src, (char*)kv_dst, g, planes, kept_pos,
                         kept_seq_offsets + num_seqs, capacity, status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return launch_status();
}
