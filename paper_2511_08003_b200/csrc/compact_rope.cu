// Stage two (b) with positional re-encoding (Section 4.1.4: the positional embedding is encoded again
// when the cache is pruned inside the LLM).  The cached keys carry a rotary embedding of their old
// position; a kept token moves from p_old = kept_pos[j] - seq_offsets[b] to p_new = j -
// kept_seq_offsets[b], so while its key row is copied it is rotated by (p_new - p_old).  Half-split
// pairing: dimension i pairs with i + rotary_dim/2, angle (p_new - p_old) * base^(-2i/rotary_dim).
// Values and the dimensions beyond rotary_dim are bit copies.
//
//   rope_table_kernel        one warp per kept row: cos / sin of its rotation angles, angles in fp64
//   kv_compact_rope_paired_kernel  (rows of a power-of-two number of vectors, at most 32) every CTA takes a
//                            contiguous run of (row tile, plane) pairs, so the cos / sin rows of a tile
//                            are staged in shared memory once and serve all planes; in a key plane the two
//                            threads of a rotary pair each load their own vector, swap it with a warp
//                            shuffle and write their own half
//   kv_compact_rope_kernel   (other shapes) the persistent (plane, tile) walk of the plain compaction; key
//                            vectors inside the rotary part also fetch their partner vector and the row's
//                            cos / sin entries (L2-resident, shared by all planes)
#include "common.cuh"
#include "compact.cuh"

#include <cuda_bf16.h>

#include <cmath>

namespace sharpv {
namespace {

constexpr int kRopeThreads = 256;
constexpr int kRopeUnroll = 4;
constexpr int kRopeCtasPerSm = 4;

struct RopeGeom {
    int64_t src_layer, src_kv, src_head, src_token;     // bytes
    int64_t dst_layer, dst_kv, dst_head, dst_token;     // bytes
    int num_kv_heads, layer_begin, row_vecs;            // row_vecs = 16-byte vectors per row
    int rot_vecs;                                       // vectors inside the rotary part (even)
    int half;                                           // rotary_dim / 2
    int64_t row_limit;                                  // rows a source plane can hold (debug range checks)
};

// cos / sin of the rotation angle of every (kept row, rotary pair).  The angle (row's move * base^(-2i/rotary_dim))
// is formed and reduced to [-pi, pi] in fp64 (two-constant split of 2 pi: the reduction is exact to 1e-11 for
// moves of 10^5 positions), its sine and cosine are then taken in fp32, the precision the table is stored in.
// The inverse frequencies are computed once per CTA.
__global__ void __launch_bounds__(256)
rope_table_kernel(const int32_t* __restrict__ kept_pos, const int32_t* __restrict__ kept_seq_offsets,
                  const int32_t* __restrict__ seq_offsets, int num_seqs, int64_t capacity, int half,
                  int rotary_dim, double log_base, float2* __restrict__ table) {
    extern __shared__ double inv_freq[];                // [half]: base^(-2i/rotary_dim) = exp(-(2i/rotary_dim) ln base)
    for (int i = threadIdx.x; i < half; i += 256) inv_freq[i] = exp(-2.0 * (double)i / (double)rotary_dim * log_base);
    __syncthreads();
    cudaGridDependencySynchronize();
    const int lane = threadIdx.x & 31;
    const int64_t j = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int64_t n = min((int64_t)__ldg(kept_seq_offsets + num_seqs), capacity);
    if (j >= n) return;
    const int b = upper_segment(kept_seq_offsets, num_seqs, (int)j);
    const double delta = (double)(j - __ldg(kept_seq_offsets + b)) -
                         (double)(__ldg(kept_pos + j) - __ldg(seq_offsets + b));
    constexpr double kInvTwoPi = 0.15915494309189533577;
    constexpr double kTwoPiHi = 6.283185307179586232;       // fl64(2 pi)
    constexpr double kTwoPiLo = 2.4492935982947064e-16;     // 2 pi - fl64(2 pi)
    for (int i = lane; i < half; i += 32) {
        const double ang = delta * inv_freq[i];
        const double turns = rint(ang * kInvTwoPi);
        const double r = fma(-turns, kTwoPiLo, fma(-turns, kTwoPiHi, ang));
        float sn, cs;
        sincosf((float)r, &sn, &cs);
        table[j * half + i] = make_float2(cs, sn);
    }
}

// rotates the pair of vectors (x1, x2) = (first half, second half) in place:
//   x1' = x1 c - x2 s,  x2' = x2 c + x1 s,  result rounded to the storage type
template <int DT>
__device__ __forceinline__ void rotate_pair(uint4& v1, uint4& v2, const float2* __restrict__ cs) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    float a[P], b[P], r1[P], r2[P];
    E::widen(v1, a);
    E::widen(v2, b);
#pragma unroll
    for (int e = 0; e < P; e += 2) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(cs + e));       // (c0, s0, c1, s1)
        r1[e] = fmaf(a[e], t.x, -b[e] * t.y);
        r2[e] = fmaf(b[e], t.x, a[e] * t.y);
        r1[e + 1] = fmaf(a[e + 1], t.z, -b[e + 1] * t.w);
        r2[e + 1] = fmaf(b[e + 1], t.z, a[e + 1] * t.w);
    }
    if (DT == SHARPV_BF16) {
        uint32_t w1[4], w2[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 h1 = __floats2bfloat162_rn(r1[2 * e], r1[2 * e + 1]);     // round to nearest even
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(r2[2 * e], r2[2 * e + 1]);
            w1[e] = *reinterpret_cast<const uint32_t*>(&h1);
            w2[e] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        v1 = make_uint4(w1[0], w1[1], w1[2], w1[3]);
        v2 = make_uint4(w2[0], w2[1], w2[2], w2[3]);
    } else {
        v1 = make_uint4(__float_as_uint(r1[0]), __float_as_uint(r1[1]), __float_as_uint(r1[P > 2 ? 2 : 0]),
                        __float_as_uint(r1[P > 3 ? 3 : 0]));
        v2 = make_uint4(__float_as_uint(r2[0]), __float_as_uint(r2[1]), __float_as_uint(r2[P > 2 ? 2 : 0]),
                        __float_as_uint(r2[P > 3 ? 3 : 0]));
    }
}

// Thread q of a tile owns vector vv = q % row_vecs of row q / row_vecs.  In a key plane the threads
// of the first half of the rotary part also fetch the partner vector and write both results; the
// threads of the second half have nothing to do.
template <int DT>
__global__ void __launch_bounds__(kRopeThreads)
kv_compact_rope_kernel(const char* __restrict__ src, char* __restrict__ dst, RopeGeom g, int planes,
                       const int32_t* __restrict__ kept_pos, const int32_t* __restrict__ n_kept_ptr,
                       int64_t capacity, const float2* __restrict__ table, int32_t* status_word) {
    constexpr int P = Elem<DT>::kPerVec;
    cudaGridDependencySynchronize();
    const int64_t n_all = __ldg(n_kept_ptr);
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_all > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    const int64_t n = min(n_all, capacity);
    if (n <= 0) return;
    const int tile_rows = kRopeThreads * kRopeUnroll / g.row_vecs;
    const int64_t tiles_per_plane = (n + tile_rows - 1) / tile_rows;
    const int64_t total_tiles = tiles_per_plane * planes;
    const int half_vecs = g.rot_vecs >> 1;
    const int64_t pair_bytes = (int64_t)half_vecs * 16;
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int plane = (int)(tile / tiles_per_plane);
        const int64_t row0 = (tile - plane * tiles_per_plane) * tile_rows;
        const int l = g.layer_begin + plane / (2 * g.num_kv_heads);
        const int kv = (plane / g.num_kv_heads) & 1;
        const int h = plane % g.num_kv_heads;
        const char* s = src + l * g.src_layer + kv * g.src_kv + h * g.src_head;
        char* o = dst + l * g.dst_layer + kv * g.dst_kv + h * g.dst_head;
        const int total = (int)min((int64_t)tile_rows, n - row0) * g.row_vecs;
        uint4 own[kRopeUnroll], partner[kRopeUnroll];
        int64_t off[kRopeUnroll];
        const float2* cs[kRopeUnroll];
        int role[kRopeUnroll];          // 0 copy, 1 rotate the pair, 2 nothing (partner of a pair)
#pragma unroll
        for (int u = 0; u < kRopeUnroll; ++u) {
            const int q = threadIdx.x + u * kRopeThreads;
            role[u] = 2;
            if (q < total) {
                const int rr = q / g.row_vecs, vv = q - rr * g.row_vecs;
                const int64_t j = row0 + rr;
                role[u] = (kv == 0 && vv < g.rot_vecs) ? (vv < half_vecs ? 1 : 2) : 0;
                const int64_t from = __ldg(kept_pos + j);
                if (!index_ok(from >= 0 && from < g.row_limit, status_word)) role[u] = 2;
                if (role[u] != 2) {
                    const char* row = s + from * g.src_token + (int64_t)vv * 16;
                    own[u] = ld_stream(row);
                    if (role[u] == 1) {
                        partner[u] = ld_stream(row + pair_bytes);
                        cs[u] = table + j * g.half + vv * P;
                    }
                    off[u] = j * g.dst_token + (int64_t)vv * 16;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kRopeUnroll; ++u) {
            if (role[u] == 1) {
                rotate_pair<DT>(own[u], partner[u], cs[u]);
                st_stream(o + off[u] + pair_bytes, partner[u]);
            }
            if (role[u] != 2) st_stream(o + off[u], own[u]);
        }
    }
}

// The key planes of the call, plane = layer * heads + head (the value planes are bit copies and go through
// the plain compaction kernel).  Tiles in (row tile, plane) order: tile = row_tile * planes + plane.  A
// CTA's run of tiles stays on one row tile for as long as possible, so the table rows of that tile are read
// from global memory once.
template <int DT>
__global__ void __launch_bounds__(kRopeThreads)
kv_compact_rope_paired_kernel(const char* __restrict__ src, char* __restrict__ dst, RopeGeom g, int planes,
                              const int32_t* __restrict__ kept_pos, const int32_t* __restrict__ n_kept_ptr,
                              int64_t capacity, const float2* __restrict__ table, int32_t* status_word) {
    constexpr int P = Elem<DT>::kPerVec;
    extern __shared__ __align__(16) unsigned char rope_smem[];
    float2* tab = reinterpret_cast<float2*>(rope_smem);        // [tile_rows][half]
    cudaGridDependencySynchronize();
    const int64_t n_all = __ldg(n_kept_ptr);
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_all > capacity) report(status_word, SHARPV_ERR_CAPACITY);
    const int64_t n = min(n_all, capacity);
    if (n <= 0) return;
    const int tile_rows = kRopeThreads * kRopeUnroll / g.row_vecs;
    const int64_t row_tiles = (n + tile_rows - 1) / tile_rows;
    const int64_t total_tiles = row_tiles * planes;
    const int64_t t0 = total_tiles * blockIdx.x / gridDim.x, t1 = total_tiles * (blockIdx.x + 1) / gridDim.x;
    if (t0 >= t1) return;
    const int half_vecs = g.rot_vecs >> 1;
    int64_t staged = -1;
    // where the run stands is stepped from tile to tile, not divided out again
    int64_t rt = t0 / planes;
    int plane = (int)(t0 - rt * planes);
    int li = plane / g.num_kv_heads, h = plane % g.num_kv_heads;
    constexpr int kv = 0;
    // what a thread handles in every tile: vector vv of row rr of the tile (rows do not straddle warps)
    int rr[kRopeUnroll], vv[kRopeUnroll];
#pragma unroll
    for (int u = 0; u < kRopeUnroll; ++u) {
        const int q = threadIdx.x + u * kRopeThreads;
        rr[u] = q / g.row_vecs;
        vv[u] = q - rr[u] * g.row_vecs;
    }
    for (int64_t tile = t0; tile < t1; ++tile) {
        const int64_t row0 = rt * tile_rows;
        const int rows = (int)min((int64_t)tile_rows, n - row0);
        if (kv == 0 && g.half > 0 && staged != rt) {            // block-uniform
            __syncthreads();                                    // nobody reads the old rows any more
            // A thread later reads the P/2 entries (two pairs each) of its own vector, the threads of a row
            // side by side: entry k of vector c of row r goes to (r * P/2 + k) * half_vecs + c, so that
            // the half_vecs threads read neighbouring 16-byte words.
            const float4* from = reinterpret_cast<const float4*>(table + row0 * g.half);
            float4* to = reinterpret_cast<float4*>(tab);
            const int per_row = g.half / 2;                     // 16-byte entries per row = half_vecs * P/2
            for (int i = threadIdx.x; i < rows * per_row; i += kRopeThreads) {
                const int r = i / per_row, m = i - r * per_row;
                const int c = m / (P / 2), k = m - c * (P / 2);
                to[(r * (P / 2) + k) * half_vecs + c] = __ldg(from + i);
            }
            __syncthreads();
            staged = rt;
        }
        const char* s = src + (g.layer_begin + li) * g.src_layer + kv * g.src_kv + h * g.src_head;
        char* o = dst + (g.layer_begin + li) * g.dst_layer + kv * g.dst_kv + h * g.dst_head;
        uint4 own[kRopeUnroll];
        int64_t off[kRopeUnroll];
#pragma unroll
        for (int u = 0; u < kRopeUnroll; ++u) {
            own[u] = make_uint4(0u, 0u, 0u, 0u);
            off[u] = -1;
            if (rr[u] < rows) {
                const int64_t j = row0 + rr[u];
                const int64_t from = __ldg(kept_pos + j);
                if (index_ok(from >= 0 && from < g.row_limit, status_word)) {
                    own[u] = ld_stream(s + from * g.src_token + (int64_t)vv[u] * 16);
                    off[u] = j * g.dst_token + (int64_t)vv[u] * 16;
                }
            }
        }
        if (kv == 0 && g.half > 0) {
#pragma unroll
            for (int u = 0; u < kRopeUnroll; ++u) {
                // the partner vector of the pair sits half_vecs lanes away
                uint4 other;
                other.x = __shfl_xor_sync(0xffffffffu, own[u].x, half_vecs);
                other.y = __shfl_xor_sync(0xffffffffu, own[u].y, half_vecs);
                other.z = __shfl_xor_sync(0xffffffffu, own[u].z, half_vecs);
                other.w = __shfl_xor_sync(0xffffffffu, own[u].w, half_vecs);
                if (off[u] >= 0 && vv[u] < g.rot_vecs) {
                    const bool second = vv[u] >= half_vecs;
                    const float4* cs = reinterpret_cast<const float4*>(tab) + rr[u] * (P / 2) * half_vecs +
                                       (vv[u] - (second ? half_vecs : 0));
                    const float sgn = second ? 1.f : -1.f;      // x1' = x1 c - x2 s,  x2' = x2 c + x1 s
                    float a[P], b[P], r[P];
                    Elem<DT>::widen(own[u], a);
                    Elem<DT>::widen(other, b);
#pragma unroll
                    for (int e = 0; e < P; e += 2) {
                        const float4 t = cs[(e / 2) * half_vecs];                       // (c0, s0, c1, s1)
                        r[e] = fmaf(a[e], t.x, b[e] * (sgn * t.y));
                        r[e + 1] = fmaf(a[e + 1], t.z, b[e + 1] * (sgn * t.w));
                    }
                    if (DT == SHARPV_BF16) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 hh = __floats2bfloat162_rn(r[2 * e], r[2 * e + 1]);
                            w[e] = *reinterpret_cast<const uint32_t*>(&hh);
                        }
                        own[u] = make_uint4(w[0], w[1], w[2], w[3]);
                    } else {
                        own[u] = make_uint4(__float_as_uint(r[0]), __float_as_uint(r[1]), __float_as_uint(r[P > 2 ? 2 : 0]),
                                            __float_as_uint(r[P > 3 ? 3 : 0]));
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kRopeUnroll; ++u)
            if (off[u] >= 0) st_stream(o + off[u], own[u]);
        if (++plane == planes) {
            plane = 0;
            ++rt;
            li = 0; h = 0;
        } else if (++h == g.num_kv_heads) {
            h = 0;
            ++li;
        }
    }
}

bool rope_layout_ok(const sharpv_kv_layout* L) {
    return L && L->num_layers >= 1 && L->num_kv_heads >= 1 && L->head_dim >= 1 && L->stride_layer >= 0 &&
           L->stride_kv >= 0 && L->stride_head >= 0 && L->stride_token >= L->head_dim;
}

bool rope_layout_aligned(const sharpv_kv_layout* L) {
    const int64_t eb = elem_bytes(L->dtype);
    return (L->head_dim * eb) % 16 == 0 && (L->stride_layer * eb) % 16 == 0 && (L->stride_kv * eb) % 16 == 0 &&
           (L->stride_head * eb) % 16 == 0 && (L->stride_token * eb) % 16 == 0;
}

}  // namespace
}  // namespace sharpv

using namespace sharpv;

extern "C" size_t sharpv_kv_compact_rope_workspace_bytes(int64_t capacity, int32_t rotary_dim) {
    if (capacity <= 0 || rotary_dim <= 0) return 256;
    return align_up((size_t)capacity * (size_t)(rotary_dim / 2) * sizeof(float2), 256);
}

extern "C" sharpv_status sharpv_kv_compact_rope(
    const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst, const sharpv_kv_layout* dst_layout,
    int32_t layer_begin, int32_t layer_end, const int32_t* kept_pos, const int32_t* kept_seq_offsets,
    const int32_t* seq_offsets, int32_t num_seqs, int64_t capacity, int32_t rotary_dim, double rope_base,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    if (!rope_layout_ok(src_layout) || !rope_layout_ok(dst_layout)) return SHARPV_ERR_INVALID_ARG;
    if (!dtype_ok(src_layout->dtype) || !dtype_ok(dst_layout->dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (src_layout->dtype != dst_layout->dtype || src_layout->head_dim != dst_layout->head_dim ||
        src_layout->num_kv_heads != dst_layout->num_kv_heads || src_layout->num_layers != dst_layout->num_layers)
        return SHARPV_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > src_layout->num_layers || layer_begin > layer_end || num_seqs < 1 ||
        capacity < 0 || rotary_dim < 0 || rotary_dim > src_layout->head_dim || (rotary_dim & 1) ||
        !(rope_base > 0.0))
        return SHARPV_ERR_INVALID_ARG;
    if (!kv_src || !kv_dst || !kept_seq_offsets || !seq_offsets || kv_src == kv_dst) return SHARPV_ERR_INVALID_ARG;
    if (capacity > 0 && !kept_pos) return SHARPV_ERR_INVALID_ARG;
    const int64_t eb = elem_bytes(src_layout->dtype);
    if (!rope_layout_aligned(src_layout) || !rope_layout_aligned(dst_layout) || !aligned16(kv_src) ||
        !aligned16(kv_dst) || ((int64_t)(rotary_dim / 2) * eb) % 16)
        return SHARPV_ERR_UNSUPPORTED;
    if (capacity >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    const int planes = (layer_end - layer_begin) * 2 * src_layout->num_kv_heads;
    if (planes == 0 || capacity == 0) return SHARPV_OK;
    if (kv_ranges_overlap(kv_src, src_layout, kv_dst, dst_layout, layer_begin, layer_end, capacity))
        return SHARPV_ERR_INVALID_ARG;
    if (rotary_dim > 0 && (!workspace || !aligned16(workspace))) return SHARPV_ERR_INVALID_ARG;
    if (workspace_bytes < sharpv_kv_compact_rope_workspace_bytes(capacity, rotary_dim)) return SHARPV_ERR_WORKSPACE;

    RopeGeom g;
    g.src_layer = src_layout->stride_layer * eb; g.src_kv = src_layout->stride_kv * eb;
    g.src_head = src_layout->stride_head * eb;   g.src_token = src_layout->stride_token * eb;
    g.dst_layer = dst_layout->stride_layer * eb; g.dst_kv = dst_layout->stride_kv * eb;
    g.dst_head = dst_layout->stride_head * eb;   g.dst_token = dst_layout->stride_token * eb;
    g.num_kv_heads = src_layout->num_kv_heads;
    g.layer_begin = layer_begin;
    g.row_vecs = (int)(src_layout->head_dim * eb / 16);
    g.rot_vecs = (int)((int64_t)rotary_dim * eb / 16);
    g.half = rotary_dim / 2;
    g.row_limit = kv_row_limit(src_layout);
    if (g.row_vecs > kRopeThreads * kRopeUnroll) return SHARPV_ERR_UNSUPPORTED;      // rows over 8 KB
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    float2* table = (float2*)workspace;
    if (rotary_dim > 0) {
        if (launch_dependent(rope_table_kernel, dim3((unsigned)((capacity + 7) / 8)), dim3(256),
                             (size_t)g.half * sizeof(double), stream, kept_pos,
                             kept_seq_offsets, seq_offsets, (int)num_seqs, capacity, g.half, (int)rotary_dim,
                             log(rope_base), table) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    const int tile_rows = kRopeThreads * kRopeUnroll / g.row_vecs;
    const int64_t max_tiles = (capacity + tile_rows - 1) / tile_rows * planes;
    const int64_t want = (int64_t)sms * kRopeCtasPerSm;
    const unsigned grid = (unsigned)(max_tiles < want ? max_tiles : want);
    // rows of a power-of-two number of vectors that fit a warp, rotary halves of a power-of-two number of
    // vectors: the two threads of a pair sit in one warp and swap their vectors with a shuffle
    const int half_vecs = g.rot_vecs / 2;
    const bool pow2_row = (g.row_vecs & (g.row_vecs - 1)) == 0 && g.row_vecs <= 32;
    const bool pow2_half = half_vecs == 0 || (half_vecs & (half_vecs - 1)) == 0;
    const size_t tab_bytes = (size_t)tile_rows * g.half * sizeof(float2);
    if (pow2_row && pow2_half && g.rot_vecs == 2 * half_vecs && tab_bytes <= 96 * 1024) {
        auto kern = src_layout->dtype == SHARPV_F32 ? kv_compact_rope_paired_kernel<SHARPV_F32>
                                                     : kv_compact_rope_paired_kernel<SHARPV_BF16>;
        if (tab_bytes > 48 * 1024 &&
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tab_bytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
        // keys here, values (half of the bytes, no arithmetic) through the plain compaction kernel
        const int key_planes = planes / 2;
        const int64_t key_tiles = (capacity + tile_rows - 1) / tile_rows * key_planes;
        const unsigned key_grid = (unsigned)(key_tiles < want ? key_tiles : want);
        if (launch_dependent(kern, dim3(key_grid), dim3(kRopeThreads), tab_bytes, stream, (const char*)kv_src,
                             (char*)kv_dst, g, key_planes, kept_pos, kept_seq_offsets + num_seqs, capacity,
                             (const float2*)table, status_word) != cudaSuccess) {
            (void)cudaGetLastError();
            return SHARPV_ERR_CUDA;
        }
        return kv_compact_launch(kv_src, src_layout, kv_dst, dst_layout, layer_begin, layer_end, kept_pos,
                                 kept_seq_offsets + num_seqs, 0, 0, capacity, status_word, stream, 1);
    }
    auto kern = src_layout->dtype == SHARPV_F32 ? kv_compact_rope_kernel<SHARPV_F32>
                                                 : kv_compact_rope_kernel<SHARPV_BF16>;
    if (launch_dependent(kern, dim3(grid), dim3(kRopeThreads), 0, stream, (const char*)kv_src, (char*)kv_dst, g,
                         planes, kept_pos, kept_seq_offsets + num_seqs, capacity, (const float2*)table,
                         status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
}
