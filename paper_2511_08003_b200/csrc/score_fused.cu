// Stage one (a) with one HBM read per token (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// The token matrix is cut into column slices of 256 bytes.  A work unit is (slice s, frame t):
// the f x 256-byte tile of frame t.  Persistent CTAs (one per SM) each take a contiguous range of
// units in (slice-major, frame-minor) order, so a CTA walks consecutive frames of one slice.
//
//   score_pass_kernel      512 threads in two roles that meet at hardware barriers:
//       row warps (up to 12; 16 lanes per row, one 16-byte vector per lane, two rows per warp
//                          and visit) keep the frame they saw last in registers, already widened
//                          to fp32, and the vectors of the next tile on their way in from global
//                          memory (one 128-bit streaming load per row and lane, issued a whole
//                          tile ahead).  A tile is visited once: each element is widened once and
//                          feeds ||a||^2, the column sums of the tile and ||a - b||^2 against the
//                          registers, which it then replaces.  While the helper turns the column
//                          sums into the frame mean the warp adds up its row sums over the 16
//                          lanes of a row (through its own patch of shared memory); then it takes
//                          <a, mean> from the registers and writes one record of partial sums per
//                          row and slice.
//       helper warps (4)   add up the column sums the row warps leave in shared memory, publish
//                          the slice of the frame mean and tell the row warps what the next unit is.
//       No thread ever spins: the roles wait for each other at bar.sync only.
//   score_finalize_kernel  one CTA per frame, launched as a programmatic dependent so that its
//       start-up overlaps the tail of the pass: adds the slices in a fixed order and writes
//       S, T, I, the ratio and the budget of the frame.
#include "score_common.cuh"
#include "score_fused.cuh"

namespace sharpv {
namespace {

constexpr int kSliceBytes = 256;
constexpr int kMaxRowWarps = 12;        // a row warp = 2 rows x 16 lanes (one vector per lane)
constexpr int kHelpWarps = 4;
constexpr int kRowThreads = kMaxRowWarps * 32;      // three warpgroups; warps beyond W stay idle
constexpr int kHelpThreads = kHelpWarps * 32;
constexpr int kThreads = kRowThreads + kHelpThreads;
constexpr int kMaxVisits = 11;          // rows a half warp keeps in registers
constexpr int kMaxTokensFused = 256;    // the finaliser takes one row per thread of a 256-thread group
static_assert(2 * kMaxRowWarps * kMaxVisits >= kMaxTokensFused, "the row warps must cover the largest frame");
constexpr int kFinThreads = 1024;

struct FusedParams {
    const char* tokens;
    int64_t row_bytes_ld;
    int F, f, d, nsl, nvec;
    int num_videos;
    const int32_t* video_frame_offsets;
    float w;
    int one_minus_cos, round_mode, min_keep;
    float *out_I, *out_S, *out_T, *out_ratio;
    int32_t* out_k;
    float* mean;            // [F, d]
    float4* part;           // [F, nsl, f]: (||a||^2, <a, m>, ||a-b||^2, ||b||^2) of the slice
    int W;                  // row warps at work: a tile is covered in R = ceil(f / 2W) visits
};

// Hardware barriers between the roles: the side that hands something over arrives, the side that
// needs it syncs; `threads` counts both sides.  A warp that waits here issues nothing meanwhile.
constexpr int kBarSums = 1;     // column sums of a tile are in colp (row warps -> helper warps)
constexpr int kBarMean = 2;     // frame mean of a tile and the next unit's tag are out (helper -> row warps)
__device__ __forceinline__ void bar_arrive(int id, int threads) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Two fp32 values in one 64-bit register, the operand form of the packed fp32 instructions.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float hsum(f32x2 v) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// one word of two bf16 -> the two exact fp32 values as a pair (a bf16 is the upper half of an fp32);
// plain integer code, so that the compiler places the halves of the pair itself
__device__ __forceinline__ f32x2 widen_bf16x2(uint32_t w) {
    return ((unsigned long long)(w & 0xffff0000u) << 32) | (unsigned long long)(w << 16);
}
__device__ __forceinline__ f32x2 pair_f32(uint32_t lo, uint32_t hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}

__device__ __forceinline__ bool frame_is_first(const int32_t* vfo, int num_videos, int t) {
    const int b = upper_segment(vfo, num_videos, t);
    return __ldg(vfo + b) == t;
}

// where a CTA stands in its range of units
struct Walk {
    int s, t;           // slice and frame of the current unit
    int vid, next_start;
    bool is_first;      // frame t opens a video

    __device__ __forceinline__ void start(const FusedParams& p, int64_t u0) {
        s = (int)(u0 / p.F);
        t = (int)(u0 % p.F);
        vid = upper_segment(p.video_frame_offsets, p.num_videos, t);
        is_first = __ldg(p.video_frame_offsets + vid) == t;
        next_start = __ldg(p.video_frame_offsets + vid + 1);
    }
    // advances to the next unit; returns true when it starts a new slice
    __device__ __forceinline__ bool step(const FusedParams& p) {
        if (++t == p.F) {
            t = 0;
            ++s;
            vid = upper_segment(p.video_frame_offsets, p.num_videos, 0);
            next_start = __ldg(p.video_frame_offsets + vid + 1);
            is_first = true;
            return true;
        }
        is_first = false;
        while (t >= next_start && vid + 1 < p.num_videos) {         // skips videos without frames
            ++vid;
            is_first = true;
            next_start = __ldg(p.video_frame_offsets + vid + 1);
        }
        return false;
    }
};


// Shared memory of one CTA (about 40 KB).
template <int DT>
struct Smem {
    static constexpr int SE = kSliceBytes / Elem<DT>::kBytes;   // elements per slice row
    static constexpr int kRedStride = 66;                       // floats per visit slot: a float2 per lane, and 2 so that the slots start on different banks
    static constexpr int kRedFloats = 16 * kRedStride;          // per row warp: 16 visit slots
    float colp[2 * kMaxRowWarps * SE];      // column sums of each half warp, lane-major order
    float red[kMaxRowWarps * kRedFloats];   // row sums of each warp on their way across lanes
    float mean_s[SE];                       // frame-mean slice of the newest tile, same order as colp
    int2 info[2];                           // of unit n, at n & 1: t * nsl + s, "opens a video"
};

// Order of the SE floats of a slice row in colp / mean_s: float 4k + q of lane j's vector sits at
// (16k + j) * 4 + q, so that the 16 lanes of a row store and load whole float4s side by side.
// Returns the column of the slice that position `off` holds.
template <int DT>
__device__ __forceinline__ int column_of_position(int off) {
    constexpr int P = Elem<DT>::kPerVec;
    const int q = off & 3, j = (off >> 2) & 15, k = off >> 6;
    return j * P + 4 * k + q;
}

template <int DT>
__device__ __forceinline__ void widen_pairs(const uint4& v, f32x2 (&o)[Elem<DT>::kPerVec / 2]) {
    constexpr int H = Elem<DT>::kPerVec / 2;
    if (DT == SHARPV_BF16) {
        o[0] = widen_bf16x2(v.x); o[1] = widen_bf16x2(v.y);
        o[H - 2] = widen_bf16x2(v.z); o[H - 1] = widen_bf16x2(v.w);
    } else {
        o[0] = pair_f32(v.x, v.y); o[H - 1] = pair_f32(v.z, v.w);
    }
}

// ---------------------------------------------------------------------------------------
// helper warps: frame mean, unit tags
// ---------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void helper_role(const FusedParams& p, Smem<DT>& sm, int64_t u0, int n_units, int htid) {
    constexpr int SE = Smem<DT>::SE;
    Walk w;
    w.start(p, u0);
    const int column = column_of_position<DT>(htid & (SE - 1));
    float* mean_out = p.mean + (int64_t)w.t * p.d + w.s * SE + column;
    const float* my_col = sm.colp + htid;
    const int groups = 2 * p.W;
    const int both = 32 * p.W + kHelpThreads;
    const float ff = (float)p.f;
    if (htid == 0) sm.info[0] = make_int2(w.t * p.nsl + w.s, w.is_first ? 1 : 0);
    bar_arrive(kBarMean, both);                 // the first unit's tag is out
    for (int n = 0; n < n_units; ++n) {
        float* out = mean_out;
        if (w.step(p)) mean_out = p.mean + w.s * SE + column;
        else mean_out += p.d;
        if (htid == 0) sm.info[(n + 1) & 1] = make_int2(w.t * p.nsl + w.s, w.is_first ? 1 : 0);
        bar_sync(kBarSums, both);
        if (htid < SE) {
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
            int gidx = 0;
#pragma unroll 2
            for (; gidx + 3 < groups; gidx += 4) {
                s0 += my_col[(gidx + 0) * SE];
                s1 += my_col[(gidx + 1) * SE];
                s2 += my_col[(gidx + 2) * SE];
                s3 += my_col[(gidx + 3) * SE];
            }
            if (gidx < groups) {            // groups is even
                s0 += my_col[(gidx + 0) * SE];
                s1 += my_col[(gidx + 1) * SE];
            }
            const float m = ((s0 + s1) + (s2 + s3)) / ff;
            sm.mean_s[htid] = m;
            *out = m;
        }
        bar_arrive(kBarMean, both);
    }
}

// ---------------------------------------------------------------------------------------
// row warps
// ---------------------------------------------------------------------------------------
// Lane (g, j) of warp `warp` (g = lane / 16) owns, in visit v, vector j of row 2 W v + 2 warp + g.
// Visits below R - 1 exist for every warp and every lane; in the last one a warp takes part if its
// first row exists, and a half warp whose own row lies beyond the frame loads nothing and works on
// zeros.
//
// Row sums cross the 16 lanes of a row through the warp's own patch of shared memory: every lane
// leaves its parts there, then lane l adds up the 16 parts of row l / 16, visit l % 16 of the warp,
// in lane order.
template <int DT, int R>
struct RowRegs {
    static constexpr int H = Elem<DT>::kPerVec / 2;
    static constexpr int kRS = 66;      // floats per visit slot of the warp's patch (Smem::kRedStride)
    f32x2 prev[R][H];       // the frame seen last, fp32 pairs: [visit][pair]
    uint4 raw[R];           // the tile about to be visited, as it arrives from global memory

    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int v = 0; v < R; ++v) {
            raw[v] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int i = 0; i < H; ++i) prev[v][i] = pk(0.f, 0.f);
        }
    }

    // requests this lane's vectors of the tile at `tile` (this lane's first row and column)
    __device__ __forceinline__ void request(const char* tile, int64_t vstride, bool last_mine) {
#pragma unroll
        for (int v = 0; v < R; ++v)
            if (v < R - 1 || last_mine) raw[v] = __ldcs(reinterpret_cast<const uint4*>(tile + v * vstride));
    }

    // One visit of the tile in `raw`: ||a||^2 and ||a - b||^2 (TEMPORAL, b = the rows in registers)
    // of this lane's part of each row go to the warp's patch, col += a (COLS), the registers then
    // hold the new rows, and the vectors of the tile behind it (`next`, if any) are requested as
    // soon as a register is free for them.
    template <bool TEMPORAL, bool COLS>
    __device__ __forceinline__ void take_tile(const char* next, int64_t vstride, bool last_warp, bool last_mine,
                                              f32x2 (&col)[H], float* red_lane) {
#pragma unroll
        for (int v = 0; v < R; ++v) {
            if (v < R - 1 || last_warp) {
                f32x2 a2[H];
                widen_pairs<DT>(raw[v], a2);
                if (next && (v < R - 1 || last_mine)) raw[v] = __ldcs(reinterpret_cast<const uint4*>(next));
                next += vstride;
                f32x2 aa, db;
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    aa = i == 0 ? mul2(a2[i], a2[i]) : fma2(a2[i], a2[i], aa);
                    if (COLS) col[i] = (v == 0 && R > 1) ? a2[i] : add2(col[i], a2[i]);
                    if (TEMPORAL) {
                        const f32x2 e = sub2(a2[i], prev[v][i]);
                        db = i == 0 ? mul2(e, e) : fma2(e, e, db);
                    }
                    prev[v][i] = a2[i];
                }
                *reinterpret_cast<float2*>(red_lane + v * kRS) = make_float2(hsum(aa), TEMPORAL ? hsum(db) : 0.f);
            }
        }
    }

    // <a, mean> of the rows in registers, this lane's part of each row, to the warp's patch
    __device__ __forceinline__ void against_mean(const f32x2 (&m)[H], bool last_warp, int g, float* red_lane) const {
#pragma unroll
        for (int v = 0; v < R; ++v) {
            if (v < R - 1 || last_warp) {
                f32x2 am;
#pragma unroll
                for (int i = 0; i < H; ++i) am = i == 0 ? mul2(prev[v][i], m[i]) : fma2(prev[v][i], m[i], am);
                red_lane[v * kRS + g] = hsum(am);
            }
        }
    }
};

template <int DT, int R>
__device__ __forceinline__ void row_role(const FusedParams& p, Smem<DT>& sm, int64_t u0, int n_units, int halo,
                                         int tid) {
    constexpr int H = Elem<DT>::kPerVec / 2, SE = Smem<DT>::SE;
    static_assert(H >= 2, "two accumulators per sum");
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 4, j = lane & 15;
    const int row0 = 2 * warp + g;
    const bool last_warp = 2 * p.W * (R - 1) + 2 * warp < p.f;      // the warp takes part in the last visit
    const bool last_mine = 2 * p.W * (R - 1) + row0 < p.f;          // and this lane's own row exists there
    const int64_t vstride = (int64_t)2 * p.W * p.row_bytes_ld;
    const int64_t frame_bytes = (int64_t)p.f * p.row_bytes_ld;
    float* my_colp = sm.colp + (2 * warp + g) * SE + j * 4;         // float4 k of this lane at + 64 k
    const float* my_mean = sm.mean_s + j * 4;
    float* red_warp = sm.red + warp * Smem<DT>::kRedFloats;
    float* red_lane = red_warp + lane * 2;                          // visit v of this lane at + 64 v
    // the row sums this lane adds up: row sg of the warp's two, visit sv, starting with lane srot
    const int sg = lane >> 4, sv = lane & 15;
    const float* sum_src = red_warp + sv * Smem<DT>::kRedStride + sg * 32;    // float2 of lane j' of the row at + 2 j'
    const int my_row = 2 * p.W * sv + 2 * warp + sg;
    const bool sums = sv < R;
    const bool writes = sums && my_row < p.f;
    const int both = 32 * p.W + kHelpThreads;

    RowRegs<DT, R> st;
    st.clear();
    float prev_aa = 0.f;            // ||row||^2 of the frame seen last, for the row this lane adds up

    // this lane's first vector of the first tile: the frame in front of the range, if it matters
    const int s0 = (int)(u0 / p.F);
    int t = (int)(u0 % p.F) - halo;
    const char* tile = p.tokens + ((int64_t)t * p.f + row0) * p.row_bytes_ld + (int64_t)s0 * kSliceBytes + j * 16;
    st.request(tile, vstride, last_mine);
    bar_sync(kBarMean, both);                   // the first unit's tag
    const int Q = n_units + halo;
    int n = 0;
    for (int q = 0; q < Q; ++q) {
        const bool halo_tile = halo && q == 0;
        // the tile behind this one: the next frame of the slice, or the first frame of the next slice
        const char* next = nullptr;
        if (q + 1 < Q) {
            if (++t == p.F) {
                t = 0;
                next = tile - (int64_t)(p.F - 1) * frame_bytes + kSliceBytes;
            } else {
                next = tile + frame_bytes;
            }
        }
        const int2 inf = sm.info[n & 1];
        const bool temporal = !halo_tile && inf.y == 0;     // the frame continues a video
        f32x2 col[H];
        if (R == 1) {               // the only visit may be one this warp has no part in
#pragma unroll
            for (int i = 0; i < H; ++i) col[i] = pk(0.f, 0.f);
        }
        if (halo_tile) st.template take_tile<false, false>(next, vstride, last_warp, last_mine, col, red_lane);
        else if (temporal) st.template take_tile<true, true>(next, vstride, last_warp, last_mine, col, red_lane);
        else st.template take_tile<false, true>(next, vstride, last_warp, last_mine, col, red_lane);
        tile = next;
        if (!halo_tile) {
#pragma unroll
            for (int k = 0; k < H / 2; ++k)
                *reinterpret_cast<ulonglong2*>(my_colp + 64 * k) = make_ulonglong2(col[2 * k], col[2 * k + 1]);
            bar_arrive(kBarSums, both);                     // the column sums are out
        }
        __syncwarp();
        // row sums of ||a||^2 and ||a - b||^2 while the helper makes the mean
        f32x2 xy = pk(0.f, 0.f);
        if (sums) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                xy = add2(xy, *reinterpret_cast<const f32x2*>(sum_src + 2 * i));
        }
        __syncwarp();                                       // the patch is free again
        float my_aa, my_db;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(my_aa), "=f"(my_db) : "l"(xy));

        if (!halo_tile) {
            bar_sync(kBarMean, both);
            f32x2 m[H];
#pragma unroll
            for (int k = 0; k < H / 2; ++k) {
                const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(my_mean + 64 * k);
                m[2 * k] = x.x;
                m[2 * k + 1] = x.y;
            }
            st.against_mean(m, last_warp, g, red_lane);
            __syncwarp();
            float my_am = 0.f;
            if (sums) {
#pragma unroll
                for (int i = 0; i < 16; ++i) my_am += sum_src[2 * i + sg];
            }
            __syncwarp();                                   // the patch is free again
            if (writes)
                p.part[(int64_t)inf.x * p.f + my_row] = make_float4(my_aa, my_am, my_db, temporal ? prev_aa : 0.f);
            ++n;
        }
        prev_aa = my_aa;
    }
}

template <int DT, int R>
__global__ void __launch_bounds__(kThreads, 1)
score_pass_kernel(const FusedParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    Smem<DT>& sm = *reinterpret_cast<Smem<DT>*>(smem);

    cudaGridDependencySynchronize();        // the tokens come from earlier work on the stream
    // Let the finaliser's CTAs be scheduled as soon as SMs free up; they wait for this whole grid.
    // Only after the wait above: what the finaliser reads before its own wait (the frame table) is
    // then known to be complete.
    cudaTriggerProgrammaticLaunchCompletion();
    const int64_t U = (int64_t)p.nsl * p.F;
    const int64_t u0 = U * blockIdx.x / gridDim.x;
    const int64_t u1 = U * (blockIdx.x + 1) / gridDim.x;
    if (u0 >= u1) return;
    const int n_units = (int)(u1 - u0);
    const int t0 = (int)(u0 % p.F);
    const int vid0 = upper_segment(p.video_frame_offsets, p.num_videos, t0);
    const int halo = (__ldg(p.video_frame_offsets + vid0) == t0) ? 0 : 1;

    // The block is launched with 128 registers per thread (512 x 128 = 65536).  The helper warps give
    // most of theirs back and the three row warpgroups take them: 128 x 32 + 384 x 160 = 65536.
    const int tid = threadIdx.x;
    if (tid < kRowThreads) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 160;");
        if ((tid >> 5) < p.W) row_role<DT, R>(p, sm, u0, n_units, halo, tid);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 32;");
        helper_role<DT>(p, sm, u0, n_units, tid - kRowThreads);
    }
}

// One CTA per frame: adds the slices in a fixed order, writes S, T, I, ratio_t and k_t.
// 1024 threads = 4 groups x 256 rows; group q adds slices q, q+4, ... (all loads in flight at once),
// then the four group sums are added in order.
template <int DT>
__global__ void __launch_bounds__(kFinThreads)
score_finalize_kernel(const FusedParams p) {
    __shared__ float4 g_sum[4][kMaxTokensFused];
    __shared__ float f_s2[kMaxTokensFused], f_t2[kMaxTokensFused], f_aa[kMaxTokensFused], f_bb[kMaxTokensFused];
    __shared__ int f_fl[kMaxTokensFused];
    __shared__ float red[kFinThreads / 32];
    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = tid & (kMaxTokensFused - 1), grp = tid >> 8;
    const bool is_first = frame_is_first(p.video_frame_offsets, p.num_videos, t);
    // everything the pass kernel wrote is visible after this point
    cudaGridDependencySynchronize();

    // every load of this thread is issued before the first one is used: one memory round trip
    const float* mean = p.mean + (int64_t)t * p.d;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float sm = 0.f;
    const float4* src = p.part + ((int64_t)t * p.nsl) * p.f + row;
    for (int s0 = grp; s0 < p.nsl; s0 += 32) {
        float4 q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int s = s0 + 4 * i;
            q[i] = (row < p.f && s < p.nsl) ? __ldcg(src + (int64_t)s * p.f) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (s0 == grp) {
            for (int c = tid * 4; c < p.d; c += kFinThreads * 4) {
                const float4 m = __ldcg(reinterpret_cast<const float4*>(mean + c));
                sm = fmaf(m.x, m.x, sm); sm = fmaf(m.y, m.y, sm); sm = fmaf(m.z, m.z, sm); sm = fmaf(m.w, m.w, sm);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) { acc.x += q[i].x; acc.y += q[i].y; acc.z += q[i].z; acc.w += q[i].w; }
    }
    g_sum[grp][row] = acc;
    sm = warp_sum(sm);
    if (lane == 0) red[warp] = sm;
    __syncthreads();
    float smm = 0.f;
#pragma unroll
    for (int i = 0; i < kFinThreads / 32; ++i) smm += red[i];

    if (tid < p.f) {
        const float4 a0 = g_sum[0][tid], a1 = g_sum[1][tid], a2 = g_sum[2][tid], a3 = g_sum[3][tid];
        const float aa = (a0.x + a1.x) + (a2.x + a3.x), am = (a0.y + a1.y) + (a2.y + a3.y);
        const float db = (a0.z + a1.z) + (a2.z + a3.z), bb = (a0.w + a1.w) + (a2.w + a3.w);
        const float s2 = dissim_sq_from_dot(aa, smm, am);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);
        int fl = 0;
        if (s2 < kRefineBelowDot) fl |= 1;
        if (!is_first && t2 < kRefineBelow && db != 0.f) fl |= 2;
        f_s2[tid] = s2; f_t2[tid] = t2; f_aa[tid] = aa; f_bb[tid] = bb; f_fl[tid] = fl;
    }
    __syncthreads();
    // nearly parallel rows: exact re-evaluation from the rows themselves (rare)
    for (int r = warp; r < p.f; r += kFinThreads / 32) {
        const int fl = f_fl[r];
        if (fl) {
            const char* pa = p.tokens + ((int64_t)t * p.f + r) * p.row_bytes_ld;
            const char* pb = pa - (int64_t)p.f * p.row_bytes_ld;
            const float ia = 1.f / fmaxf(sqrtf(f_aa[r]), kNormEps);
            const float ib = 1.f / fmaxf(sqrtf(f_bb[r]), kNormEps);
            const float im = 1.f / fmaxf(sqrtf(smm), kNormEps);
            float es, et;
            refine_row<DT>(pa, pb, mean, p.nvec, lane, (fl & 1) != 0, (fl & 2) != 0, ia, ib, im, es, et);
            if (lane == 0) {
                if (fl & 1) f_s2[r] = es;
                if (fl & 2) f_t2[r] = et;
            }
        }
    }
    __syncthreads();
    float tsq = 0.f;
    if (tid < p.f) {
        float S, T, I;
        scores_from_sq(f_s2[tid], f_t2[tid], is_first, p.one_minus_cos, p.w, S, T, I);
        const int64_t o = (int64_t)t * p.f + tid;
        p.out_I[o] = I;
        if (p.out_S) p.out_S[o] = S;
        if (p.out_T) p.out_T[o] = T;
        tsq = T * T;
    }
    tsq = warp_sum(tsq);
    if (lane == 0) red[warp] = tsq;         // rows live in the first 8 warps; the others add zeros
    __syncthreads();
    if (tid == 0) {
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < kFinThreads / 32; ++i) tot += red[i];
        const float r = ratio_from_sumsq(tot, p.f);
        p.out_ratio[t] = r;
        p.out_k[t] = budget_from_ratio(r, p.f, p.round_mode, p.min_keep);
    }
}

// The split of a frame over the row warps: W warps cover 2W rows a visit and the frame in
// R = ceil(f / 2W) visits; warp w sits on scheduler w mod 4.  The split with the lightest
// busiest scheduler wins, then the larger W.
void row_split(int f, int& W, int& R) {
    int best = 1 << 30;
    W = kMaxRowWarps;
    R = kMaxVisits;
    for (int w = 1; w <= kMaxRowWarps; ++w) {
        const int r = (f + 2 * w - 1) / (2 * w);
        if (r > kMaxVisits) continue;
        int load[4] = {0, 0, 0, 0};
        for (int i = 0; i < w; ++i) load[i & 3] += r - 1 + (2 * w * (r - 1) + 2 * i < f ? 1 : 0);
        int worst = 0;
        for (int k = 0; k < 4; ++k) worst = load[k] > worst ? load[k] : worst;
        if (worst <= best) { best = worst; W = w; R = r; }
    }
}

template <int DT, int R>
sharpv_status launch(const FusedScoreArgs& a, FusedParams& p, int sms) {
    const size_t smem = sizeof(Smem<DT>);
    if (cudaFuncSetAttribute(score_pass_kernel<DT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_UNSUPPORTED;
    }
    const int64_t units = (int64_t)p.nsl * a.F;
    const unsigned grid = (unsigned)(units < sms ? units : sms);
    if (launch_dependent(score_pass_kernel<DT, R>, dim3(grid), dim3(kThreads), smem, a.stream, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
#ifdef NOFIN
    return SHARPV_OK;
#endif
    // the finaliser starts while the pass drains and waits for it with cudaGridDependencySynchronize
    if (launch_dependent(score_finalize_kernel<DT>, dim3((unsigned)a.F), dim3(kFinThreads), 0, a.stream, p) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
}

template <int DT>
sharpv_status launch_visits(const FusedScoreArgs& a, FusedParams& p, int sms, int R) {
    switch (R) {
        case 1: return launch<DT, 1>(a, p, sms);
        case 2: return launch<DT, 2>(a, p, sms);
        case 3: return launch<DT, 3>(a, p, sms);
        case 4: return launch<DT, 4>(a, p, sms);
        case 5: return launch<DT, 5>(a, p, sms);
        case 6: return launch<DT, 6>(a, p, sms);
        case 7: return launch<DT, 7>(a, p, sms);
        case 8: return launch<DT, 8>(a, p, sms);
        case 9: return launch<DT, 9>(a, p, sms);
        case 10: return launch<DT, 10>(a, p, sms);
        case 11: return launch<DT, 11>(a, p, sms);
    }
    return SHARPV_ERR_UNSUPPORTED;
}

}  // namespace

bool fused_score_supported(sharpv_dtype dtype, int f, int d) {
    const int64_t row_bytes = (int64_t)d * elem_bytes(dtype);
    return f >= 1 && f <= kMaxTokensFused && row_bytes % kSliceBytes == 0;
}

size_t fused_score_workspace_bytes(int F, int f, int d) {
    const size_t nsl_max = ((size_t)d * 4 + kSliceBytes - 1) / kSliceBytes;
    return align_up((size_t)F * d * 4, 256) + align_up((size_t)F * nsl_max * f * 16, 256);
}

sharpv_status fused_score_launch(const FusedScoreArgs& a) {
    const int eb = elem_bytes(a.dtype);
    FusedParams p;
    p.tokens = (const char*)a.tokens;
    p.row_bytes_ld = a.ld_tokens * eb;
    p.F = a.F; p.f = a.f; p.d = a.d;
    p.nsl = (int)((int64_t)a.d * eb / kSliceBytes);
    p.nvec = a.d * eb / 16;
    p.num_videos = a.num_videos;
    p.video_frame_offsets = a.video_frame_offsets;
    p.w = a.w; p.one_minus_cos = a.one_minus_cos; p.round_mode = a.round_mode; p.min_keep = a.min_keep;
    p.out_I = a.out_I; p.out_S = a.out_S; p.out_T = a.out_T; p.out_ratio = a.out_ratio; p.out_k = a.out_k;
    char* w = (char*)a.workspace;
    p.mean = (float*)w;       w += align_up((size_t)a.F * a.d * 4, 256);
    p.part = (float4*)w;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    int R = 0;
    row_split(a.f, p.W, R);
    return a.dtype == SHARPV_F32 ? launch_visits<SHARPV_F32>(a, p, sms, R)
                                 : launch_visits<SHARPV_BF16>(a, p, sms, R);
}

}  // namespace sharpv
