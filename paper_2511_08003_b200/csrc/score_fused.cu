// Stage one (a) with one HBM read per token (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// The token matrix is cut into column slices of 128 bytes.  A work unit is (slice s, frame t): the
// f x 128-byte tile of frame t.  Every CTA takes a contiguous run of units in (slice-major,
// frame-minor) order, so it walks consecutive frames of one slice; several CTAs share an SM and
// cover each other's waits.
//
//   score_pass_kernel   Up to 8 warps; a warp covers 4 rows per visit (8 lanes per row, one 16-byte
//       vector per lane) and a tile in R visits.  A thread owns the same (row, vector) positions in
//       every tile of the run:
//         - the tile it saw last stays, as stored, in the thread's own slots of shared memory,
//         - the tile it is about to see is on its way from global memory into registers (128-bit
//           streaming loads issued a whole tile ahead).
//       One visit per tile: the new vector a and the stored vector b of the frame in front are
//       widened once and feed ||a||^2, the column sums of the tile, ||a - b||^2 and <b, mean of b's
//       frame> (the mean term of a tile is taken one tile late, when its column sums have become the
//       frame mean, so no warp waits for the mean inside a tile).  Row sums cross the 8 lanes of a row
//       through the warp's own patch of shared memory.  Per row and slice three partial sums go to
//       the workspace.  Two block barriers per tile; nothing polls.
//       The kernel never looks at the video table: the temporal partial sum of a frame that opens a
//       video is computed against whatever tile was in front and ignored by the finaliser.
//   score_finalize_kernel  one CTA per frame, launched as a programmatic dependent so that its
//       start-up overlaps the tail of the pass: adds the slices in a fixed order and writes
//       S, T, I, the ratio and the budget of the frame.
#include "score_common.cuh"
#include "score_fused.cuh"

namespace sharpv {
namespace {

constexpr int kSliceBytes = 128;
constexpr int kMaxWarps = 8;            // a warp = 4 rows x 8 lanes (one vector per lane) per visit
constexpr int kMaxVisits = 8;           // rows a lane group walks per tile
constexpr int kMaxTokensFused = 256;    // the finaliser takes one row per thread of a 256-thread group
static_assert(4 * kMaxWarps * kMaxVisits >= kMaxTokensFused, "the warps must cover the largest frame");
constexpr int kRedStride = 9;           // floats per (visit, row) slot of a warp's patch: 8 lane parts + 1 pad

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
    float4* part;           // [F, nsl, f]: (||a||^2, <a, mean>, ||a-b||^2, ||b||^2) of the row's part in the slice,
                            // b = the same position one frame earlier
    int32_t* kept_local;    // [F, f] or null: the finaliser also selects; frame t's kept tokens (ascending) at t * f
    int W;                  // warps per CTA: a tile is covered in R = ceil(f / 4W) visits
    int32_t* status_word;   // may be null
};

constexpr int kBarSums = 1;     // the column sums of a tile are in shared memory
constexpr int kBarMean = 2;     // the frame-mean slice of a tile is in shared memory
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
__device__ __forceinline__ void unpk(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ float hsum(f32x2 v) {
    float lo, hi;
    unpk(v, lo, hi);
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

template <int DT> struct Pairs;
template <> struct Pairs<SHARPV_BF16> {
    static constexpr int H = 4;     // fp32 pairs per 16-byte vector
    __device__ __forceinline__ static void widen(const uint4& v, f32x2 (&o)[4]) {
        o[0] = widen_bf16x2(v.x); o[1] = widen_bf16x2(v.y); o[2] = widen_bf16x2(v.z); o[3] = widen_bf16x2(v.w);
    }
};
template <> struct Pairs<SHARPV_F32> {
    static constexpr int H = 2;
    __device__ __forceinline__ static void widen(const uint4& v, f32x2 (&o)[2]) {
        o[0] = pair_f32(v.x, v.y); o[1] = pair_f32(v.z, v.w);
    }
};

__device__ __forceinline__ f32x2 shfl_xor2(f32x2 v, int mask) {
    float lo, hi;
    unpk(v, lo, hi);
    lo = __shfl_xor_sync(0xffffffffu, lo, mask);
    hi = __shfl_xor_sync(0xffffffffu, hi, mask);
    return pk(lo, hi);
}


__device__ __forceinline__ bool frame_is_first(const int32_t* vfo, int num_videos, int t) {
    const int b = upper_segment(vfo, num_videos, t);
    return __ldg(vfo + b) == t;
}

// Shared memory of one CTA of W warps and R visits, in this order:
//   float2 red2[W][4 R * 9]       per warp: lane parts of (||a||^2, ||a-b||^2)
//   float  red1[W][4 R * 9]       per warp: lane parts of <b, mean>
//   float  colp[W][SE]            per warp: column sums of the tile
//   float  mean_s[SE]             frame-mean slice of the newest tile
constexpr size_t pass_smem_bytes(int W, int R, int SE) {
    return (size_t)W * 4 * R * kRedStride * 12 + (size_t)W * SE * 4 + (size_t)SE * 4;
}

template <int DT, int R>
__global__ void __launch_bounds__(32 * kMaxWarps, 2)
score_pass_kernel(const FusedParams p) {
    constexpr int H = Pairs<DT>::H;
    constexpr int P = Elem<DT>::kPerVec;
    constexpr int SE = kSliceBytes / Elem<DT>::kBytes;      // elements per slice row
    constexpr int kPlane = 4 * R * kRedStride;              // slots of a warp's patch
    constexpr int D = R >= 6 ? 1 : 0;                     // visits by which the hand-over of a register lags
    extern __shared__ __align__(16) unsigned char smem[];

    const int W = p.W, NT = 32 * W;
    float2* red2 = reinterpret_cast<float2*>(smem);
    float* red1 = reinterpret_cast<float*>(red2 + W * kPlane);
    float* colp = red1 + W * kPlane;
    float* mean_s = colp + W * SE;

    cudaGridDependencySynchronize();        // the tokens come from earlier work on the stream
    // Let the finaliser's CTAs be scheduled as soon as SMs free up; they wait for this whole grid.
    cudaTriggerProgrammaticLaunchCompletion();
    const int64_t U = (int64_t)p.nsl * p.F;
    const int64_t u0 = U * blockIdx.x / gridDim.x;
    const int64_t u1 = U * (blockIdx.x + 1) / gridDim.x;
    if (u0 >= u1) return;
    const int n_units = (int)(u1 - u0);
    int s = (int)(u0 / p.F), t = (int)(u0 % p.F);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 3, j = lane & 7;
    const int row0 = 4 * warp + g;                                  // this lane's row in visit 0
    const bool last_mine = (R - 1) * 4 * W + row0 < p.f;            // its row of the last visit exists
    const bool last_warp = (R - 1) * 4 * W + 4 * warp < p.f;        // the warp has a row in the last visit
    const int64_t vstride = (int64_t)4 * W * p.row_bytes_ld;
    const int64_t frame_bytes = (int64_t)p.f * p.row_bytes_ld;
    float2* red2_lane = red2 + warp * kPlane + g * kRedStride + j;  // visit v at + 4 v * kRedStride
    float* red1_lane = red1 + warp * kPlane + g * kRedStride + j;
    // the row sums this lane adds up: visit sv, row sg of the warp's four
    const int sv = lane >> 2, sg = lane & 3;
    const float2* sum2_src = red2 + warp * kPlane + lane * kRedStride;
    const float* sum1_src = red1 + warp * kPlane + lane * kRedStride;
    const int my_row = sv * 4 * W + 4 * warp + sg;
    const bool sums = sv < R;
    const bool writes = sums && my_row < p.f;
    const int mean_warps = W < SE / 32 ? W : SE / 32;               // warps that turn column sums into the mean
    const float inv_f = 1.f / (float)p.f;

    // Two tiles live in registers as stored: the one being visited and the one in front of it.  The
    // registers of the one in front are handed, vector by vector, to the tile behind, so the names
    // swap from tile to tile and nothing is copied.
    uint4 ta[R], tb[R];
    const char* nxt = p.tokens + ((int64_t)t * p.f + row0) * p.row_bytes_ld + (int64_t)s * kSliceBytes + j * 16;
#pragma unroll
    for (int v = 0; v < R; ++v) {
        const bool mine = v < R - 1 || last_mine;
        ta[v] = make_uint4(0u, 0u, 0u, 0u);
        tb[v] = make_uint4(0u, 0u, 0u, 0u);
        if (mine) ta[v] = __ldcs(reinterpret_cast<const uint4*>(nxt + v * vstride));
        if (mine && t > 0) tb[v] = __ldcs(reinterpret_cast<const uint4*>(nxt - frame_bytes + v * vstride));
    }

    f32x2 m[H];                     // this lane's columns of the mean of the frame in front
#pragma unroll
    for (int i = 0; i < H; ++i) m[i] = pk(0.f, 0.f);
    int t_prev = t, s_prev = s;

    // What the lane that adds up a row keeps from tile to tile: ||a||^2 and ||a-b||^2 of the tile seen
    // last (its record is written one tile late, together with its mean term) and that tile's ||b||^2,
    // which is the ||a||^2 of the tile before it.  For the first tile of the run that is the frame in
    // front of the run, still in `tb`.
    float keep_aa = 0.f, keep_db = 0.f, keep_bb = 0.f;
    if (t > 0) {
#pragma unroll
        for (int v = 0; v < R; ++v) {
            f32x2 b2[H];
            Pairs<DT>::widen(tb[v], b2);
            f32x2 bb;
#pragma unroll
            for (int i = 0; i < H; ++i) bb = i == 0 ? mul2(b2[i], b2[i]) : fma2(b2[i], b2[i], bb);
            red1_lane[4 * v * kRedStride] = hsum(bb);
        }
        __syncwarp();
        if (sums) {
            float x = sum1_src[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) x += sum1_src[i];
            keep_aa = x;
        }
        __syncwarp();
    }

    // One tile: `cur` is visited against `old`; the registers of `old` receive the tile behind `cur`.
    auto visit_tile = [&](uint4 (&cur)[R], uint4 (&old)[R], int n) {
        // the tile behind this one: the next frame of the slice, or the first frame of the next slice
        const bool has_next = n + 1 < n_units;
        int t_next = t + 1, s_next = s;
        if (t_next == p.F) {
            t_next = 0;
            s_next = s + 1;
            nxt += kSliceBytes - (int64_t)(p.F - 1) * frame_bytes;
        } else {
            nxt += frame_bytes;
        }
        const char* q = nxt;

        f32x2 col[H];
#pragma unroll
        for (int v = 0; v < R; ++v) {
            const bool active = v < R - 1 || R == 1 || last_warp;   // warp-uniform
            f32x2 a2[H], b2[H];
            if (active) {
                Pairs<DT>::widen(cur[v], a2);
                Pairs<DT>::widen(old[v], b2);
            }
            if (v >= D) {
                if (has_next && (v - D < R - 1 || last_mine)) old[v - D] = __ldcs(reinterpret_cast<const uint4*>(q));
                q += vstride;
            }
            if (active) {
                f32x2 aa, db, bm;
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    aa = i == 0 ? mul2(a2[i], a2[i]) : fma2(a2[i], a2[i], aa);
                    col[i] = v == 0 ? a2[i] : add2(col[i], a2[i]);
                    const f32x2 e = sub2(a2[i], b2[i]);
                    db = i == 0 ? mul2(e, e) : fma2(e, e, db);
                    bm = i == 0 ? mul2(b2[i], m[i]) : fma2(b2[i], m[i], bm);
                }
                red2_lane[4 * v * kRedStride] = make_float2(hsum(aa), hsum(db));
                red1_lane[4 * v * kRedStride] = hsum(bm);
            }
        }
#pragma unroll
        for (int v = R - D; v < R; ++v) {
            if (v >= 0) {
                if (has_next && (v < R - 1 || last_mine)) old[v] = __ldcs(reinterpret_cast<const uint4*>(q));
                q += vstride;
            }
        }
        // column sums of the warp's four row groups, then one partial per warp
#pragma unroll
        for (int i = 0; i < H; ++i) {
            col[i] = add2(col[i], shfl_xor2(col[i], 8));
            col[i] = add2(col[i], shfl_xor2(col[i], 16));
        }
        if (lane < 8) {
            float* dst = colp + warp * SE + lane * P;
#pragma unroll
            for (int i = 0; i < H; i += 2)
                *reinterpret_cast<ulonglong2*>(dst + 2 * i) = make_ulonglong2(col[i], col[i + 1]);
        }
        if (warp >= mean_warps) bar_arrive(kBarSums, NT);
        __syncwarp();
        // row sums over the 8 lanes of a row
        if (sums) {
            f32x2 x2 = *reinterpret_cast<const f32x2*>(sum2_src);
            float xm = sum1_src[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) {
                x2 = add2(x2, *reinterpret_cast<const f32x2*>(sum2_src + i));
                xm += sum1_src[i];
            }
            float xa, xd;
            unpk(x2, xa, xd);
            if (writes && n > 0 && index_ok(t_prev < p.F && s_prev < p.nsl, p.status_word))
                p.part[((int64_t)t_prev * p.nsl + s_prev) * p.f + my_row] = make_float4(keep_aa, xm, keep_db, keep_bb);
            keep_bb = keep_aa;
            keep_aa = xa;
            keep_db = xd;
        }
        if (warp < mean_warps) {
            bar_sync(kBarSums, NT);
            float* mean_out = p.mean + (int64_t)t * p.d + s * SE;
            for (int c = tid; c < SE; c += 32 * mean_warps) {
                float acc = colp[c];
                for (int q2 = 1; q2 < W; ++q2) acc += colp[q2 * SE + c];
                acc *= inv_f;
                mean_s[c] = acc;
                mean_out[c] = acc;
            }
        }
        bar_sync(kBarMean, NT);
        {
            const float* src = mean_s + j * P;
#pragma unroll
            for (int i = 0; i < H; i += 2) {
                const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(src + 2 * i);
                m[i] = x.x;
                m[i + 1] = x.y;
            }
        }
        t_prev = t;
        s_prev = s;
        t = t_next;
        s = s_next;
    };

    // the mean term of the last tile of the run
    auto last_mean_term = [&](const uint4 (&last)[R]) {
#pragma unroll
        for (int v = 0; v < R; ++v) {
            f32x2 b2[H];
            Pairs<DT>::widen(last[v], b2);
            f32x2 bm;
#pragma unroll
            for (int i = 0; i < H; ++i) bm = i == 0 ? mul2(b2[i], m[i]) : fma2(b2[i], m[i], bm);
            red1_lane[4 * v * kRedStride] = hsum(bm);
        }
        __syncwarp();
        if (writes && index_ok(t_prev < p.F && s_prev < p.nsl, p.status_word)) {
            float xm = sum1_src[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) xm += sum1_src[i];
            p.part[((int64_t)t_prev * p.nsl + s_prev) * p.f + my_row] = make_float4(keep_aa, xm, keep_db, keep_bb);
        }
    };

    int n = 0;
    for (; n + 1 < n_units; n += 2) {
        visit_tile(ta, tb, n);
        visit_tile(tb, ta, n + 1);
    }
    if (n < n_units) {
        visit_tile(ta, tb, n);
        last_mean_term(ta);
    } else {
        last_mean_term(tb);
    }
}

// One CTA per frame: adds the slices in a fixed order, writes S, T, I, ratio_t and k_t.
// G groups of 256 rows; group q adds slices q, q+G, ... (up to 8 records in flight per thread), then the
// group sums are added in order.  G = 4 (1024 threads, one CTA on an SM) is the quickest for a frame;
// G = 2 (512 threads, two CTAs on an SM) takes twice the frames at a time and is used when there are
// more frames than SMs.
template <int DT, int G>
__global__ void __launch_bounds__(256 * G, G == 2 ? 2 : 0)
score_finalize_kernel(const FusedParams p) {
    constexpr int kFinThreads = 256 * G;
    __shared__ float4 g_sum[G][kMaxTokensFused];
    __shared__ float f_all[4 * kMaxTokensFused];        // four per-row arrays, later the four partial ranks
    float* const f_s2 = f_all;
    float* const f_t2 = f_all + kMaxTokensFused;
    float* const f_aa = f_all + 2 * kMaxTokensFused;
    float* const f_bb = f_all + 3 * kMaxTokensFused;
    __shared__ int f_fl[kMaxTokensFused];
    __shared__ float red[kFinThreads / 32 + 1];     // also the scratch of the block scan
    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = tid & (kMaxTokensFused - 1), grp = tid >> 8;
    const bool is_first = frame_is_first(p.video_frame_offsets, p.num_videos, t);
    // everything the pass kernel wrote is visible after this point
    cudaGridDependencySynchronize();

    const float* mean = p.mean + (int64_t)t * p.d;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);       // ||a||^2, <a, mean>, ||a - b||^2, ||b||^2
    float sm = 0.f;
    const float4* src = p.part + ((int64_t)t * p.nsl) * p.f + row;
    for (int s0 = grp; s0 < p.nsl; s0 += 8 * G) {
        float4 q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int s = s0 + G * i;
            q[i] = (row < p.f && s < p.nsl) ? __ldcg(src + (int64_t)s * p.f) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (s0 == grp) {
            for (int c = tid * 4; c < p.d; c += kFinThreads * 4) {
                const float4 mm = __ldcg(reinterpret_cast<const float4*>(mean + c));
                sm = fmaf(mm.x, mm.x, sm); sm = fmaf(mm.y, mm.y, sm); sm = fmaf(mm.z, mm.z, sm); sm = fmaf(mm.w, mm.w, sm);
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
        float aa, am, db, bb;
        if constexpr (G == 4) {
            const float4 a0 = g_sum[0][tid], a1 = g_sum[1][tid], a2 = g_sum[2][tid], a3 = g_sum[3][tid];
            aa = (a0.x + a1.x) + (a2.x + a3.x); am = (a0.y + a1.y) + (a2.y + a3.y);
            db = (a0.z + a1.z) + (a2.z + a3.z); bb = (a0.w + a1.w) + (a2.w + a3.w);
        } else {
            const float4 a0 = g_sum[0][tid], a1 = g_sum[1][tid];
            aa = a0.x + a1.x; am = a0.y + a1.y; db = a0.z + a1.z; bb = a0.w + a1.w;
        }
        const float s2 = dissim_sq_from_dot(aa, smm, am);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);      // a video's first frame: db, bb unused
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
    float tsq = 0.f, my_I = 0.f;
    if (tid < p.f) {
        float S, T, I;
        scores_from_sq(f_s2[tid], f_t2[tid], is_first, p.one_minus_cos, p.w, S, T, I);
        my_I = I;
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
        const int kt = budget_from_ratio(r, p.f, p.round_mode, p.min_keep);
        p.out_ratio[t] = r;
        p.out_k[t] = kt;
        f_fl[0] = kt;
    }
    if (!p.kept_local) return;

    // Per-frame top-k (Section 3.1.3, last paragraph) while the frame's scores are still here: a token's
    // rank under (score descending, index ascending) is the number of composite (key, ~index) keys above
    // its own; it is kept iff rank < k_t.  The kept tokens go, ascending, to the frame's staging row.
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(&g_sum[0][0]);   // the slice sums are spent
    __syncthreads();                        // k_t is out, g_sum is free
    const int kt = f_fl[0];
    unsigned long long mine = ~0ull;
    if (tid < kMaxTokensFused) {
        if (tid < p.f) mine = ((unsigned long long)order_key(my_I) << 32) | (0xffffffffu - (uint32_t)tid);
        comp[tid] = tid < p.f ? mine : 0ull;
    }
    __syncthreads();
    // all groups of 256 threads count: group q compares token `row` with the keys q, q+G, ... of the
    // frame (as pairs), the partial ranks meet in shared memory
    int* ranks = reinterpret_cast<int*>(f_all);         // [G][256]; the per-row arrays were last read barriers ago
    const unsigned long long my_key = row < p.f ? comp[row] : ~0ull;
    {
        int part = 0;
        const int fpad = (p.f + 1) & ~1;
        for (int j2 = 2 * grp; j2 < fpad; j2 += 2 * G) {
            const ulonglong2 c2 = *reinterpret_cast<const ulonglong2*>(comp + j2);
            part += (c2.x > my_key) + (c2.y > my_key);
        }
        ranks[grp * kMaxTokensFused + row] = part;
    }
    __syncthreads();
    int keep = 0;
    if (tid < p.f && kt > 0) {
        int rank = ranks[tid] + ranks[kMaxTokensFused + tid];
        if constexpr (G == 4) rank += ranks[2 * kMaxTokensFused + tid] + ranks[3 * kMaxTokensFused + tid];
        keep = rank < kt;
    }
    int total;
    const int pos = block_exclusive_scan<kFinThreads>(keep, reinterpret_cast<int*>(red), total);
    if (keep) p.kept_local[(int64_t)t * p.f + pos] = tid;
}

// Second half of the single-call stage one: the kept lists of the frames become one ascending list of
// global token indices, and the kept rows are copied (Section 3.1: the retained tokens form the pruned
// visual sequence).  Persistent CTAs; every CTA first scans the budgets (up to kEmitInlineFrames
// frames; beyond, a scan kernel in front has left the offsets in kept_offsets), then takes half rows
// in a grid-stride loop: one warp per half row, 128-bit copies.
constexpr int kEmitThreads = 256;
constexpr int kEmitInlineFrames = 4096;

__global__ void __launch_bounds__(kEmitThreads)
emit_gather_kernel(const int32_t* __restrict__ k, const int32_t* __restrict__ kept_local, int F, int f,
                   int offsets_ready, int32_t* __restrict__ kept_offsets, int32_t* __restrict__ num_kept,
                   int32_t* __restrict__ out_kept_index, int64_t capacity, const char* __restrict__ src,
                   int64_t src_row_bytes, int nvec, char* __restrict__ dst, int64_t dst_row_bytes,
                   int32_t* status_word) {
    __shared__ int32_t off_s[kEmitInlineFrames + 1];
    __shared__ int scan_sm[kEmitThreads / 32 + 1];
    const int tid = threadIdx.x, lane = tid & 31;
    cudaGridDependencySynchronize();        // budgets and kept lists come from the kernel in front
    int64_t n_total;
    if (!offsets_ready) {
        // exclusive scan of the clamped budgets: thread i owns a contiguous share
        const int per = (F + kEmitThreads - 1) / kEmitThreads;
        const int lo = min(F, tid * per), hi = min(F, lo + per);
        int sum = 0;
        for (int i = lo; i < hi; ++i) sum += min(max(k[i], 0), f);
        int total;
        int run = block_exclusive_scan<kEmitThreads>(sum, scan_sm, total);
        for (int i = lo; i < hi; ++i) {
            off_s[i] = run;
            run += min(max(k[i], 0), f);
        }
        if (tid == 0) off_s[F] = total;
        __syncthreads();
        n_total = total;
        if (blockIdx.x == 0) {
            for (int i = tid; i <= F; i += kEmitThreads) kept_offsets[i] = off_s[i];
            if (tid == 0) {
                if (num_kept) *num_kept = total;
                if ((int64_t)total > capacity) report(status_word, SHARPV_ERR_CAPACITY);
            }
        }
    } else {
        n_total = kept_offsets[F];
    }
    const int64_t n = min(n_total, capacity);
    const int half = (nvec + 1) >> 1;
    for (int64_t w = (int64_t)blockIdx.x * (kEmitThreads / 32) + (tid >> 5); w < 2 * n;
         w += (int64_t)gridDim.x * (kEmitThreads / 32)) {
        const int64_t j = w >> 1;
        const int t = offsets_ready ? upper_segment(kept_offsets, F, (int)j) : upper_segment_any(off_s, F, (int)j);
        const int base = offsets_ready ? __ldg(kept_offsets + t) : off_s[t];
        const int32_t local = __ldg(kept_local + (int64_t)t * f + (j - base));
        if (!index_ok(j - base < f && local >= 0 && local < f, status_word)) continue;
        const int32_t row_index = t * f + local;
        if ((w & 1) == 0 && lane == 0) out_kept_index[j] = row_index;
        if (!dst) continue;
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
}

// The split of a frame over the warps of a CTA: W warps of 4 rows a visit, R = ceil(f / 4W) visits.
// The split with the fewest warp-visits wins (no warp idles through a visit), then the one with
// fewer visits.
void row_split(int f, int& W, int& R) {
    int best = 1 << 30;
    W = kMaxWarps;
    R = kMaxVisits;
    for (int w = 1; w <= kMaxWarps; ++w) {
        const int r = (f + 4 * w - 1) / (4 * w);
        if (r > kMaxVisits) continue;
        if (w * r < best || (w * r == best && r < R)) { best = w * r; W = w; R = r; }
    }
}

template <int DT, int R>
sharpv_status launch(const FusedScoreArgs& a, FusedParams& p, int dev, int sms) {
    constexpr int SE = kSliceBytes / Elem<DT>::kBytes;
    auto kernel = score_pass_kernel<DT, R>;
    const size_t smem = pass_smem_bytes(p.W, R, SE);
    // resident CTAs per SM of this instance and block size, asked once per device
    static int resident[64][kMaxWarps + 1] = {};
    if (dev < 0 || dev >= 64) return SHARPV_ERR_UNSUPPORTED;
    int per_sm = resident[dev][p.W];
    if (per_sm == 0) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)pass_smem_bytes(kMaxWarps, R, SE)) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 32 * p.W, smem) != cudaSuccess ||
            per_sm < 1) {
            (void)cudaGetLastError();
            return SHARPV_ERR_UNSUPPORTED;
        }
        resident[dev][p.W] = per_sm;
    }
    const int64_t units = (int64_t)p.nsl * a.F;
    const int64_t slots = (int64_t)sms * per_sm;
    const unsigned grid = (unsigned)(units < slots ? units : slots);
    if (launch_dependent(kernel, dim3(grid), dim3(32 * p.W), smem, a.stream, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    // the finaliser starts while the pass drains and waits for it with cudaGridDependencySynchronize
    const cudaError_t fin = a.F > sms
        ? launch_dependent(score_finalize_kernel<DT, 2>, dim3((unsigned)a.F), dim3(512), 0, a.stream, p)
        : launch_dependent(score_finalize_kernel<DT, 4>, dim3((unsigned)a.F), dim3(1024), 0, a.stream, p);
    if (fin != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    if (!a.select) return SHARPV_OK;

    // single-call stage one: offsets of the frames' kept lists, one global list, the kept rows
    const int offsets_ready = a.F > kEmitInlineFrames;
    if (offsets_ready &&
        launch_dependent(exclusive_scan_i32_kernel<true>, dim3(1), dim3(kScanThreads), 0, a.stream,
                         (const int32_t*)a.out_k, (int64_t)a.F, (int)a.f, a.out_kept_offsets, a.out_kept_offsets + a.F,
                         a.out_num_kept, a.capacity, a.status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    const int64_t rows = a.capacity < (int64_t)a.F * a.f ? a.capacity : (int64_t)a.F * a.f;
    const int64_t want = (2 * rows + kEmitThreads / 32 - 1) / (kEmitThreads / 32);
    const int64_t most = (int64_t)sms * 8;
    const unsigned egrid = (unsigned)(want < 1 ? 1 : (want < most ? want : most));
    if (launch_dependent(emit_gather_kernel, dim3(egrid), dim3(kEmitThreads), 0, a.stream, (const int32_t*)a.out_k,
                         (const int32_t*)p.kept_local, (int)a.F, (int)a.f, offsets_ready, a.out_kept_offsets,
                         a.out_num_kept, a.out_kept_index, a.capacity, (const char*)a.tokens, p.row_bytes_ld, p.nvec,
                         (char*)a.out_tokens, (int64_t)a.d * elem_bytes(a.dtype), a.status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
}

template <int DT>
sharpv_status launch_visits(const FusedScoreArgs& a, FusedParams& p, int dev, int sms, int R) {
    switch (R) {
        case 1: return launch<DT, 1>(a, p, dev, sms);
        case 2: return launch<DT, 2>(a, p, dev, sms);
        case 3: return launch<DT, 3>(a, p, dev, sms);
        case 4: return launch<DT, 4>(a, p, dev, sms);
        case 5: return launch<DT, 5>(a, p, dev, sms);
        case 6: return launch<DT, 6>(a, p, dev, sms);
        case 7: return launch<DT, 7>(a, p, dev, sms);
        case 8: return launch<DT, 8>(a, p, dev, sms);
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

size_t fused_select_workspace_bytes(int F, int f) { return align_up((size_t)F * f * 4, 256); }

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
    p.status_word = a.status_word;
    char* w = (char*)a.workspace;
    p.mean = (float*)w;       w += align_up((size_t)a.F * a.d * 4, 256);
    p.part = (float4*)w;
    // the staging rows of the kept lists sit behind the largest extent the scores' scratch can have
    p.kept_local = a.select ? (int32_t*)((char*)a.workspace + fused_score_workspace_bytes(a.F, a.f, a.d)) : nullptr;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    int R = 0;
    row_split(a.f, p.W, R);
    return a.dtype == SHARPV_F32 ? launch_visits<SHARPV_F32>(a, p, dev, sms, R)
                                 : launch_visits<SHARPV_BF16>(a, p, dev, sms, R);
}

}  // namespace sharpv
