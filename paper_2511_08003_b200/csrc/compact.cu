// Stage two (b): K/V compaction (Section 3.2.3).  For every (layer, K|V, head) plane the rows
// of the kept positions are copied, in order, to a dense prefix of the destination plane.
// One index list serves all planes.
//
// Out of place: one short-lived CTA per (row tile, plane) with 128-bit loads and stores through
// registers.  In place (kv_dst == kv_src): the rows are split into levels of disjoint row ranges (below).
// Bulk async copies (one cp.async.bulk per kept 256-byte row into a shared-memory tile, one bulk
// store per dense tile) were measured and lost: the copy engine's per-request cost caps 256-byte
// rows near 2.2 TB/s of reads, against 2.7 TB/s for this kernel at the same kept share.
#include "common.cuh"
#include "compact.cuh"

namespace sharpv {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kCompactUnroll = 4;         // 16-byte vectors in flight per thread
constexpr int kCompactCtasPerSm = 5;      // resident CTAs per SM of the in-place level kernel (47 registers)
constexpr int kGatherCtasPerSm = 8;       // of the out-of-place kernel: 32 registers, every thread slot of an SM taken
constexpr int kGatherTilesPerCta = 2;     // row tiles a CTA takes at least when the list is as long as `capacity`
constexpr int64_t kGatherMaxCtas = 32768; // CTAs of one launch (many times the 148 x 8 that are resident)

struct PlaneGeom {
    int64_t src_layer, src_kv, src_head, src_token;     // bytes
    int64_t dst_layer, dst_kv, dst_head, dst_token;     // bytes
    int num_kv_heads, layer_begin, row_vecs;            // row_vecs = 16-byte vectors per row
    int row_shift;                                      // log2(row_vecs) if that is a power of two, else -1
    int64_t row_limit;                                  // rows a source plane can hold (what a dense layout implies)
};

// One CTA per (row tile, plane): tile_rows destination rows of one plane; blockIdx.y is the plane.  Each
// thread moves kUnroll 16-byte vectors, all loads issued before the first store.  The grid is laid out for
// `capacity` rows (the kept count is only known on the device) with kGatherTilesPerCta tiles to a CTA; a CTA
// whose tile starts behind the kept count leaves at once.  CTAs that come and go keep reads and writes of
// the SMs mixed: persistent CTAs walking the same tiles in step stay about 10 % under it.
template <int kUnroll, bool kPerLayer>
__global__ void __launch_bounds__(kCompactThreads, kGatherCtasPerSm)
kv_compact_kernel(const char* __restrict__ src, char* __restrict__ dst, PlaneGeom g,
                  const int32_t* __restrict__ kept_pos, const int32_t* __restrict__ n_kept_ptr,
                  int64_t kept_stride, int64_t count_stride, int64_t capacity, int kv_only, int32_t* status_word) {
    // blockIdx.y counts the planes of the call: (layer, K|V, head), or (layer, head) of the keys / the values alone
    const int plane = blockIdx.y;
    const int h = plane % g.num_kv_heads;
    const int li = kv_only < 0 ? plane / (2 * g.num_kv_heads) : plane / g.num_kv_heads;
    const int kv = kv_only < 0 ? (plane / g.num_kv_heads) & 1 : kv_only;
    const int tile_rows = kCompactThreads * kUnroll / g.row_vecs;      // >= 1, checked by the host
    cudaGridDependencySynchronize();        // the index list and the cache come from earlier work on the stream
    // One list for all layers (strides 0), or every layer of the range its own list and count.
    const int32_t* list = kPerLayer ? kept_pos + li * kept_stride : kept_pos;
    const int64_t n_all = __ldg(n_kept_ptr + (kPerLayer ? li * count_stride : 0));
    if (blockIdx.x == 0 && threadIdx.x == 0 && (kv == 0 || kv_only > 0) && h == 0 && (kPerLayer || li == 0) &&
        n_all > capacity)
        report(status_word, SHARPV_ERR_CAPACITY);
    const int64_t n = min(n_all, capacity);
    const char* s = src + (g.layer_begin + li) * g.src_layer + kv * g.src_kv + h * g.src_head;
    char* o = dst + (g.layer_begin + li) * g.dst_layer + kv * g.dst_kv + h * g.dst_head;
    // the grid holds a fraction of the row tiles `capacity` rows would need: a CTA takes tile blockIdx.x,
    // then blockIdx.x + gridDim.x, ... while they start in front of the kept count
    for (int64_t row0 = (int64_t)blockIdx.x * tile_rows; row0 < n; row0 += (int64_t)gridDim.x * tile_rows) {
        uint4 r[kUnroll];
        unsigned moved = 0;                 // bit u: vector u of this thread is copied
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int q = threadIdx.x + u * kCompactThreads;
            const int rr = g.row_shift >= 0 ? q >> g.row_shift : q / g.row_vecs;      // row of the tile, vector of the row
            const int64_t j = row0 + rr;
            if (rr < tile_rows && j < n) {
                const int64_t from = __ldg(list + j);
                if (index_ok(from >= 0 && from < g.row_limit, status_word)) {
                    r[u] = ld_stream(s + from * g.src_token + (int64_t)(q - rr * g.row_vecs) * 16);
                    moved |= 1u << u;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int q = threadIdx.x + u * kCompactThreads;
            const int rr = g.row_shift >= 0 ? q >> g.row_shift : q / g.row_vecs;
            if (moved >> u & 1) st_stream(o + (row0 + rr) * g.dst_token + (int64_t)(q - rr * g.row_vecs) * 16, r[u]);
        }
    }
}

// In-place compaction (kv_dst == kv_src).  Row j of the result comes from row kept_pos[j] >= j, so
// rows are only ever moved forward, but a row may be overwritten while another row still has to be
// read from it.  With b_0 = n (the kept count) and b_{k+1} = the first j whose source kept_pos[j] is
// at or behind b_k, the rows j in [b_{k+1}, b_k) read sources in [b_k, b_{k-1}) (behind n for k = 0)
// and write destinations in [b_{k+1}, b_k): inside such a level nothing that is read is written, so a
// level is copied by all SMs at once like the out-of-place case, and the levels only have to run
// innermost first (level k+1 reads what level k overwrites).  kInplaceLevels levels are peeled off
// that way; the rows in front of the innermost boundary are walked front to back by one CTA per
// plane: the loads of tile k+1 are issued, a block barrier orders every thread's loads of tile k
// before anybody's stores of tile k, then tile k is stored while tile k+1 is in flight.  Rows that
// stay where they are (kept_pos[j] == j) are not touched.  With a list per layer (layer-by-layer
// call) every plane is walked front to back in full.
constexpr int kInplaceThreads = 512;
constexpr int kInplaceUnroll = 4;
constexpr int kInplaceLevels = 3;

// First j in [0, n) with list[j] >= x (n if there is none), list ascending.  The whole block takes
// part (NT-ary search with __syncthreads_count); every thread returns the answer.
// With SHIFT the searched sequence is list[j] - j (how far row j moves; non-decreasing as well).
template <int NT, bool SHIFT = false>
__device__ __forceinline__ int64_t block_lower_bound(const int32_t* __restrict__ list, int64_t n, int64_t x) {
    int64_t lo = 0, hi = n;             // the answer is in [lo, hi]; list[lo - 1] < x, list[hi] >= x
    while (hi > lo) {
        const int64_t step = (hi - lo + NT - 1) / NT;
        const int64_t probe = lo + (int64_t)threadIdx.x * step;
        const int below = (probe < hi && (int64_t)__ldg(list + probe) - (SHIFT ? probe : 0) < x) ? 1 : 0;
        const int c = __syncthreads_count(below);
        if (c == 0) {
            hi = lo;
        } else {
            const int64_t last_below = lo + (int64_t)(c - 1) * step;
            hi = min(hi, lo + (int64_t)c * step);
            lo = last_below + 1;
        }
    }
    return lo;
}

// boundary b_{level}: b_0 = n, b_{k+1} = first j with kept_pos[j] >= b_k
template <int NT>
__device__ __forceinline__ void level_bounds(const int32_t* __restrict__ kept_pos, int64_t n, int level, int64_t& hi,
                                             int64_t& lo) {
    hi = n;
    lo = block_lower_bound<NT>(kept_pos, hi, hi);
    for (int k = 0; k < level; ++k) {
        hi = lo;
        lo = block_lower_bound<NT>(kept_pos, hi, hi);
    }
}

// front-to-back walk of the rows [0, b_{first_level}) of every plane (first_level < 0: all n rows)
__global__ void __launch_bounds__(kInplaceThreads)
kv_compact_inplace_kernel(char* __restrict__ kv, PlaneGeom g, const int32_t* __restrict__ kept_pos,
                          const int32_t* __restrict__ n_kept_ptr, int64_t kept_stride, int64_t count_stride,
                          int64_t capacity, int first_level, int32_t* status_word) {
    cudaGridDependencySynchronize();
    const int plane = blockIdx.x;
    const int li = plane / (2 * g.num_kv_heads);            // the layer's own list and count, if it has them
    kept_pos += li * kept_stride;
    const int64_t n_all = __ldg(n_kept_ptr + li * count_stride);
    if (plane % (2 * g.num_kv_heads) == 0 && threadIdx.x == 0 && n_all > capacity)
        report(status_word, SHARPV_ERR_CAPACITY);
    int64_t n = min(n_all, capacity);
    if (n <= 0) return;
    if (first_level >= 0) {
        int64_t hi, lo;
        level_bounds<kInplaceThreads>(kept_pos, n, first_level, hi, lo);
        n = lo;                                             // the rows behind it are copied level by level
        if (n <= 0) return;
    }
    const int l = g.layer_begin + li;
    const int kvi = (plane / g.num_kv_heads) & 1;
    const int h = plane % g.num_kv_heads;
    char* base = kv + l * g.src_layer + kvi * g.src_kv + h * g.src_head;
    const int tile_rows = kInplaceThreads * kInplaceUnroll / g.row_vecs;
    const int64_t tiles = (n + tile_rows - 1) / tile_rows;
    // the rows in front of the first one that moves stay as they are: start at its tile
    const int64_t first_tile = block_lower_bound<kInplaceThreads, true>(kept_pos, n, 1) / tile_rows;
    if (first_tile >= tiles) return;

    uint4 cur[kInplaceUnroll], nxt[kInplaceUnroll];
    bool cur_moves[kInplaceUnroll], nxt_moves[kInplaceUnroll];
    auto load_tile = [&](int64_t k, uint4 (&r)[kInplaceUnroll], bool (&moves)[kInplaceUnroll]) {
        const int64_t row0 = k * tile_rows;
        const int total = (int)min((int64_t)tile_rows, n - row0) * g.row_vecs;
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) {
            const int q = threadIdx.x + u * kInplaceThreads;
            moves[u] = false;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                const int64_t from = __ldg(kept_pos + row0 + rr);
                moves[u] = from != row0 + rr && index_ok(from > row0 + rr && from < g.row_limit, status_word);
                if (moves[u])
                    r[u] = *reinterpret_cast<const uint4*>(base + from * g.src_token + (int64_t)vv * 16);
            }
        }
    };
    load_tile(first_tile, cur, cur_moves);
    for (int64_t k = first_tile; k < tiles; ++k) {
        if (k + 1 < tiles) load_tile(k + 1, nxt, nxt_moves);
        __syncthreads();                        // every load of tile k happened before any store of tile k
        const int64_t row0 = k * tile_rows;
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) {
            const int q = threadIdx.x + u * kInplaceThreads;
            if (cur_moves[u]) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                *reinterpret_cast<uint4*>(base + (row0 + rr) * g.src_token + (int64_t)vv * 16) = cur[u];
            }
        }
#pragma unroll
        for (int u = 0; u < kInplaceUnroll; ++u) {
            cur[u] = nxt[u];
            cur_moves[u] = nxt_moves[u];
        }
    }
}

// one level [b_{level+1}, b_level) of the in-place compaction: sources and destinations are disjoint
// row ranges, so this is the persistent (plane, tile) walk of the out-of-place kernel on one cache
template <int kUnroll>
__global__ void __launch_bounds__(kCompactThreads, kCompactCtasPerSm)
kv_compact_inplace_level_kernel(char* __restrict__ kv, PlaneGeom g, int planes, const int32_t* __restrict__ kept_pos,
                                const int32_t* __restrict__ n_kept_ptr, int64_t capacity, int level,
                                int32_t* status_word) {
    cudaGridDependencySynchronize();
    const int64_t n = min((int64_t)__ldg(n_kept_ptr), capacity);
    if (n <= 0) return;
    int64_t hi, lo;
    level_bounds<kCompactThreads>(kept_pos, n, level, hi, lo);
    const int64_t rows_all = hi - lo;
    if (rows_all <= 0) return;
    const int tile_rows = kCompactThreads * kUnroll / g.row_vecs;
    const int64_t tiles_per_plane = (rows_all + tile_rows - 1) / tile_rows;
    const int64_t total_tiles = tiles_per_plane * planes;
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int plane = (int)(tile / tiles_per_plane);
        const int64_t row0 = lo + (tile - plane * tiles_per_plane) * tile_rows;
        const int l = g.layer_begin + plane / (2 * g.num_kv_heads);
        const int kvi = (plane / g.num_kv_heads) & 1;
        const int h = plane % g.num_kv_heads;
        char* base = kv + l * g.src_layer + kvi * g.src_kv + h * g.src_head;
        const int total = (int)min((int64_t)tile_rows, hi - row0) * g.row_vecs;
        uint4 r[kUnroll];
        int64_t off[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int q = threadIdx.x + u * kCompactThreads;
            off[u] = -1;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                const int64_t j = row0 + rr;
                const int64_t from = __ldg(kept_pos + j);
                if (from != j && index_ok(from >= hi && from < g.row_limit, status_word)) {
                    r[u] = ld_stream(base + from * g.src_token + (int64_t)vv * 16);
                    off[u] = j * g.src_token + (int64_t)vv * 16;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (off[u] >= 0) st_stream(base + off[u], r[u]);
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

namespace sharpv {

sharpv_status kv_compact_launch(const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst,
                                const sharpv_kv_layout* dst_layout, int32_t layer_begin, int32_t layer_end,
                                const int32_t* kept_pos, const int32_t* n_kept_ptr, int64_t kept_stride,
                                int64_t count_stride, int64_t capacity, int32_t* status_word, cudaStream_t stream,
                                int kv_only) {
    if (!layout_ok(src_layout) || !layout_ok(dst_layout)) {
        if (src_layout && dst_layout && (!copy_dtype_ok(src_layout->dtype) || !copy_dtype_ok(dst_layout->dtype)))
            return SHARPV_ERR_UNSUPPORTED;
        return SHARPV_ERR_INVALID_ARG;
    }
    if (src_layout->dtype != dst_layout->dtype || src_layout->head_dim != dst_layout->head_dim ||
        src_layout->num_kv_heads != dst_layout->num_kv_heads || src_layout->num_layers != dst_layout->num_layers)
        return SHARPV_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > src_layout->num_layers || layer_begin > layer_end || capacity < 0)
        return SHARPV_ERR_INVALID_ARG;
    if (!kv_src || !kv_dst || !n_kept_ptr || kv_only < -1 || kv_only > 1) return SHARPV_ERR_INVALID_ARG;
    const bool in_place = kv_src == kv_dst;
    if (in_place && kv_only >= 0) return SHARPV_ERR_INVALID_ARG;
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
    g.row_limit = kv_row_limit(src_layout);
    g.row_shift = -1;
    for (int b = 0; b < 31; ++b)
        if (g.row_vecs == 1 << b) g.row_shift = b;
    if (g.row_vecs > kCompactThreads * kCompactUnroll) return SHARPV_ERR_UNSUPPORTED;    // rows over 16 KB
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    const int tile_rows = kCompactThreads * kCompactUnroll / g.row_vecs;
    const int64_t max_tiles = (capacity + tile_rows - 1) / tile_rows * planes;
    const int64_t want = (int64_t)sms * kCompactCtasPerSm;
    const unsigned grid = (unsigned)(max_tiles < want ? max_tiles : want);
    if (in_place) {
        // one list for all planes: the innermost rows front to back, then the levels, innermost first
        const bool levels = count_stride == 0;
        if (launch_dependent(kv_compact_inplace_kernel, dim3((unsigned)planes), dim3(kInplaceThreads), 0, stream,
                             (char*)kv_dst, g, kept_pos, n_kept_ptr, kept_stride, count_stride, capacity,
                             levels ? kInplaceLevels - 1 : -1, status_word) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
        for (int level = kInplaceLevels - 1; levels && level >= 0; --level) {
            if (launch_dependent(kv_compact_inplace_level_kernel<kCompactUnroll>, dim3(grid), dim3(kCompactThreads), 0,
                                 stream, (char*)kv_dst, g, planes, kept_pos, n_kept_ptr, capacity, level,
                                 status_word) != cudaSuccess) {
                (void)cudaGetLastError();
                return SHARPV_ERR_CUDA;
            }
        }
        return SHARPV_OK;
    }
    auto kern = count_stride != 0 ? kv_compact_kernel<kCompactUnroll, true> : kv_compact_kernel<kCompactUnroll, false>;
    // at most kGatherMaxCtas CTAs in all: with a list much shorter than `capacity` most of them only look
    // at the count and leave, and that has to stay cheap
    int64_t row_tiles = ((capacity + tile_rows - 1) / tile_rows + kGatherTilesPerCta - 1) / kGatherTilesPerCta;
    const int64_t most = kGatherMaxCtas / planes > 1 ? kGatherMaxCtas / planes : 1;
    if (row_tiles > most) row_tiles = most;
    const int planes_here = kv_only < 0 ? planes : planes / 2;
    if (launch_dependent(kern, dim3((unsigned)row_tiles, (unsigned)planes_here), dim3(kCompactThreads), 0, stream,
                         (const char*)kv_src, (char*)kv_dst, g, kept_pos, n_kept_ptr, kept_stride,
                         count_stride, capacity, kv_only, status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
}

}  // namespace sharpv

extern "C" sharpv_status sharpv_kv_compact(
    const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst, const sharpv_kv_layout* dst_layout,
    int32_t layer_begin, int32_t layer_end, const int32_t* kept_pos, const int32_t* kept_seq_offsets,
    int32_t num_seqs, int64_t capacity, int32_t* status_word, void* cuda_stream) {
    if (num_seqs < 1) return SHARPV_ERR_INVALID_ARG;
    return kv_compact_launch(kv_src, src_layout, kv_dst, dst_layout, layer_begin, layer_end, kept_pos,
                             kept_seq_offsets ? kept_seq_offsets + num_seqs : nullptr, 0, 0, capacity, status_word,
                             (cudaStream_t)cuda_stream);
}
