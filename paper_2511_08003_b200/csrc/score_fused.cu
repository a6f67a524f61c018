// Stage one (a) with one HBM read per token (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// The token matrix is cut into column slices of 256 bytes.  A work unit is (slice s, frame t):
// the f x 256-byte tile of frame t.  Persistent CTAs (one per SM) each take a contiguous range of
// units in (slice-major, frame-minor) order, so a CTA walks consecutive frames of one slice.
//
//   score_pass_kernel      TMA brings the next tiles into a ring of shared-memory buffers.  Each
//       thread keeps its part of the previous frame's tile in registers (4 rows x two 16-byte
//       vectors) and visits the new tile once: column sums (they give this slice of the frame
//       mean, the whole frame column being inside the tile), ||a||^2, ||a-b||^2 against the
//       previous frame, and <b, mean(b)> for the previous frame, whose mean is known by now.
//       The new rows then replace the old ones in the same registers.  Per-row partial sums of
//       the slice go to a small workspace.  The only wait is on the CTA's own TMA loads and it
//       is bounded.
//   score_finalize_kernel  one CTA per frame, launched with programmatic dependent launch so that
//       its start-up overlaps the tail of the pass: adds the slices in a fixed order and writes
//       S, T, I, the ratio and the budget of the frame.
#include <cuda.h>

#include "score_common.cuh"
#include "score_fused.cuh"

namespace sharpv {
namespace {

constexpr int kSliceBytes = 256;
constexpr int kThreads = 512;           // 16 warps; a warp = 4 row groups x 8 lanes (two vectors per lane)
constexpr int kWarps = kThreads / 32;
constexpr int kRowGroups = kThreads / 8;
constexpr int kRows = 4;                // row slots per thread: frames of up to 256 tokens
constexpr int kMaxTokensFused = 256;
constexpr int kSmemBudget = 227 * 1024;
constexpr uint32_t kSpinLimit = 1u << 22;      // polls of one mbarrier before a wait gives up
constexpr int kFinThreads = 256;

struct FusedParams {
    const char* tokens;
    int64_t row_bytes_ld;
    int F, f, d, nsl, nvec, nbuf;
    int num_videos;
    const int32_t* video_frame_offsets;
    float w;
    int one_minus_cos, round_mode, min_keep;
    float *out_I, *out_S, *out_T, *out_ratio;
    int32_t* out_k;
    float* mean;            // [F, d]
    float4* part;           // [F, nsl, f]: (||a||^2, ||a-b||^2, ||b||^2, <a, mean>) of the slice
    uint32_t tile_bytes, tile_stride;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: false when the limit ran out
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// 8 lanes x 16 values (x[4*slot + j], 4 slots) -> lane L of the group ends with x[0], x[1] =
// values 2*(L&1), 2*(L&1)+1 of slot L>>1.  Fixed pairing, hence a fixed summation order.
__device__ __forceinline__ void group8_reduce_scatter(float (&x)[16], int lane8) {
    {
        const bool up = lane8 & 4;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float lo = x[i], hi = x[8 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 4);
        }
    }
    {
        const bool up = lane8 & 2;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = x[i], hi = x[4 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 2);
        }
    }
    {
        const bool up = lane8 & 1;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float lo = x[i], hi = x[2 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 1);
        }
    }
}

__device__ __forceinline__ bool frame_is_first(const int32_t* vfo, int num_videos, int t) {
    const int b = upper_segment(vfo, num_videos, t);
    return __ldg(vfo + b) == t;
}

template <int DT>
struct Pass {
    using E = Elem<DT>;
    static constexpr int P = E::kPerVec;                    // elements per 16-byte vector
    static constexpr int H = P / 2;                         // float2 pairs per vector
    static constexpr int SE = kSliceBytes / E::kBytes;      // elements per slice row

    const CUtensorMap* tmap;
    const FusedParams* p;
    unsigned char* tiles;
    float* cs;              // [kRowGroups][SE] column sums of each row group
    float* cs2;             // [4][SE]
    float* mean_s;          // [SE]
    uint64_t* bars;         // [nbuf]
    volatile int* abort_flag;
    int64_t u0;
    int Q, halo;

    // per-thread state carried from frame to frame
    uint4 prev[kRows][2];   // previous frame's rows of this thread (two vectors each)
    float2 mprev[2][H];     // previous frame's mean over this thread's columns
    float bb[kRows];        // this thread's share of ||previous row||^2

    int warp, g, j, rgid;

    __device__ __forceinline__ int row_of(int r) const { return warp + kWarps * (4 * r + g); }

    __device__ __forceinline__ void issue_load(int q) const {
        const FusedParams& pp = *p;
        const int64_t u = u0 + q - halo;
        int t, s;
        if (halo && q == 0) { s = (int)(u0 / pp.F); t = (int)(u0 % pp.F) - 1; }
        else { s = (int)(u / pp.F); t = (int)(u % pp.F); }
        uint64_t* bar = bars + (q % pp.nbuf);
        mbar_expect_tx(bar, pp.tile_bytes);
        tma_load_2d(tiles + (size_t)(q % pp.nbuf) * pp.tile_stride, tmap, s * kSliceBytes, t * pp.f, bar);
    }

    __device__ __forceinline__ const unsigned char* wait_tile(int q) const {
        const int nb = p->nbuf;
        if (!mbar_wait(bars + (q % nb), (uint32_t)((q / nb) & 1))) *abort_flag = 1;
        return tiles + (size_t)(q % nb) * p->tile_stride;
    }

    __device__ __forceinline__ static void to_pairs(const uint4& v, float2 (&o)[H]) {
        float x[P];
        E::widen(v, x);
#pragma unroll
        for (int i = 0; i < H; ++i) o[i] = make_float2(x[2 * i], x[2 * i + 1]);
    }

    // Frame in front of the first unit: registers only.
    __device__ __forceinline__ void load_halo(int q) {
        const unsigned char* tile = wait_tile(q);
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const int row = row_of(r);
            float2 acc = make_float2(0.f, 0.f);
            if (row < p->f) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    prev[r][h] = *reinterpret_cast<const uint4*>(tile + row * kSliceBytes + (j + 8 * h) * 16);
                    float2 b2[H];
                    to_pairs(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc = __ffma2_rn(b2[i], b2[i], acc);
                }
            }
            bb[r] = acc.x + acc.y;
        }
    }

    // x[4r + 3] = <previous row, previous mean> over this thread's columns (the other entries 0),
    // reduced over the row's 8 lanes and written to the previous frame's partial record.
    __device__ __forceinline__ void flush_prev(int s, int t_prev) {
        float x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = 0.f;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            if (row_of(r) < p->f) {
                float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float2 b2[H];
                    to_pairs(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc = __ffma2_rn(b2[i], mprev[h][i], acc);
                }
                x[4 * r + 3] = acc.x + acc.y;
            }
        }
        group8_reduce_scatter(x, j);
        const int row = warp + kWarps * (4 * (j >> 1) + g);
        if ((j & 1) && row < p->f) p->part[((int64_t)t_prev * p->nsl + s) * p->f + row].w = x[1];
    }

    // One unit: tile q = (slice s, frame t).
    //   has_prev  the registers hold frame t-1 of this slice
    //   own_prev  ... and it was a unit of this CTA, so its <row, mean> is computed here
    // Returns false when the CTA must stop (a bounded wait ran out).
    __device__ __forceinline__ bool unit(int q, int s, int t, bool has_prev, bool own_prev) {
        const FusedParams& pp = *p;
        const bool temporal = has_prev && !frame_is_first(pp.video_frame_offsets, pp.num_videos, t);
        const unsigned char* tile = wait_tile(q);

        float2 colsum[2][H];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < H; ++i) colsum[h][i] = make_float2(0.f, 0.f);
        float x[16];
        const float2 one = make_float2(1.f, 1.f), neg1 = make_float2(-1.f, -1.f);
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const int row = row_of(r);
            float2 aa = make_float2(0.f, 0.f), db = aa, bm = aa;
            if (row < pp.f) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 a4 = *reinterpret_cast<const uint4*>(tile + row * kSliceBytes + (j + 8 * h) * 16);
                    float2 a2[H];
                    to_pairs(a4, a2);
#pragma unroll
                    for (int i = 0; i < H; ++i) {
                        colsum[h][i] = __ffma2_rn(a2[i], one, colsum[h][i]);
                        aa = __ffma2_rn(a2[i], a2[i], aa);
                    }
                    if (has_prev) {
                        float2 b2[H];
                        to_pairs(prev[r][h], b2);
                        if (temporal) {
#pragma unroll
                            for (int i = 0; i < H; ++i) {
                                const float2 e = __ffma2_rn(b2[i], neg1, a2[i]);        // a - b
                                db = __ffma2_rn(e, e, db);
                            }
                        }
                        if (own_prev) {
#pragma unroll
                            for (int i = 0; i < H; ++i) bm = __ffma2_rn(b2[i], mprev[h][i], bm);
                        }
                    }
                    prev[r][h] = a4;
                }
            }
            x[4 * r + 0] = aa.x + aa.y;
            x[4 * r + 1] = db.x + db.y;
            x[4 * r + 2] = has_prev ? bb[r] : 0.f;
            x[4 * r + 3] = bm.x + bm.y;
            bb[r] = x[4 * r + 0];
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float* dst = cs + rgid * SE + (j + 8 * h) * P;
#pragma unroll
            for (int i = 0; i < H; i += 2)
                *reinterpret_cast<float4*>(dst + 2 * i) =
                    make_float4(colsum[h][i].x, colsum[h][i].y, colsum[h][i + 1].x, colsum[h][i + 1].y);
        }
        __syncthreads();                            // tile buffer free, column partials visible
        if (*abort_flag) return false;
        const int tid = threadIdx.x;
        if (tid == 0 && q + pp.nbuf < Q) issue_load(q + pp.nbuf);
        // column sums over the 64 row groups: fixed order, two levels
        for (int e = tid; e < 4 * SE; e += kThreads) {
            const int col = e % SE, quarter = e / SE;
            float sum = 0.f;
#pragma unroll 8
            for (int i = 0; i < kRowGroups / 4; ++i) sum += cs[(quarter * (kRowGroups / 4) + i) * SE + col];
            cs2[quarter * SE + col] = sum;
        }

        // per-row partial sums of the slice (overlaps the mean reduction of the other warps)
        group8_reduce_scatter(x, j);
        {
            const int row = warp + kWarps * (4 * (j >> 1) + g);
            if (row < pp.f) {
                float4* rec = pp.part + ((int64_t)t * pp.nsl + s) * pp.f + row;
                if (j & 1) {
                    rec->z = x[0];                                              // ||b||^2
                    if (own_prev) pp.part[((int64_t)(t - 1) * pp.nsl + s) * pp.f + row].w = x[1];
                } else {
                    *reinterpret_cast<float2*>(rec) = make_float2(x[0], x[1]);  // ||a||^2, ||a-b||^2
                }
            }
        }
        __syncthreads();
        if (tid < SE) {
            const float m = ((cs2[tid] + cs2[SE + tid]) + (cs2[2 * SE + tid] + cs2[3 * SE + tid])) / (float)pp.f;
            mean_s[tid] = m;
            pp.mean[(int64_t)t * pp.d + s * SE + tid] = m;
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < H; ++i)
                mprev[h][i] = *reinterpret_cast<const float2*>(mean_s + (j + 8 * h) * P + 2 * i);
        return true;
    }
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
score_pass_kernel(const __grid_constant__ CUtensorMap tmap, const FusedParams p, int32_t* status_word) {
    constexpr int SE = Pass<DT>::SE;
    extern __shared__ __align__(1024) unsigned char smem[];
    Pass<DT> c;
    c.tmap = &tmap;
    c.p = &p;
    c.tiles = smem;
    c.cs = reinterpret_cast<float*>(smem + (size_t)p.nbuf * p.tile_stride);
    c.cs2 = c.cs + kRowGroups * SE;
    c.mean_s = c.cs2 + 4 * SE;
    c.bars = reinterpret_cast<uint64_t*>(c.mean_s + SE);
    c.abort_flag = reinterpret_cast<volatile int*>(c.bars + 4);

    const int64_t U = (int64_t)p.nsl * p.F;
    c.u0 = U * blockIdx.x / gridDim.x;
    const int64_t u1 = U * (blockIdx.x + 1) / gridDim.x;
    // let the finaliser's CTAs be scheduled as soon as SMs free up; they wait for this whole grid
    cudaTriggerProgrammaticLaunchCompletion();
    if (c.u0 >= u1) return;
    c.halo = frame_is_first(p.video_frame_offsets, p.num_videos, (int)(c.u0 % p.F)) ? 0 : 1;
    c.Q = (int)(u1 - c.u0) + c.halo;

    const int tid = threadIdx.x, lane = tid & 31;
    c.warp = tid >> 5;
    c.g = lane >> 3;
    c.j = lane & 7;
    c.rgid = c.warp * 4 + c.g;
    if (tid == 0) {
        for (int i = 0; i < p.nbuf; ++i) mbar_init(c.bars + i, 1);
        *c.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0)
        for (int q = 0; q < p.nbuf && q < c.Q; ++q) c.issue_load(q);

#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        c.prev[r][0] = make_uint4(0u, 0u, 0u, 0u);
        c.prev[r][1] = c.prev[r][0];
        c.bb[r] = 0.f;
    }

    int q = 0;
    bool ok = true, has_prev = false, own_prev = false;
    if (c.halo) {
        c.load_halo(0);
        __syncthreads();
        ok = *c.abort_flag == 0;
        if (ok && tid == 0 && p.nbuf < c.Q) c.issue_load(p.nbuf);
        q = 1;
        has_prev = true;
    }
    int s_cur = (int)(c.u0 / p.F);
    for (int64_t u = c.u0; ok && u < u1; ++u, ++q) {
        const int s = (int)(u / p.F), t = (int)(u % p.F);
        if (s != s_cur) {                           // the range crosses into the next slice
            if (own_prev) c.flush_prev(s_cur, p.F - 1);
            has_prev = false;
            own_prev = false;
            s_cur = s;
        }
        ok = c.unit(q, s, t, has_prev, own_prev);
        has_prev = true;
        own_prev = true;
    }
    if (ok) {
        if (own_prev) c.flush_prev(s_cur, (int)((u1 - 1) % p.F));
    } else {
        // A wait on the CTA's own loads ran out.  Report it, then give the loads that are still in
        // flight one more bounded wait each, so that nothing lands in shared memory after exit.
        __syncthreads();
        if (tid == 0) {
            report(status_word, SHARPV_ERR_TIMEOUT);
            const int last = min(c.Q, q + p.nbuf);
            for (int i = q; i < last; ++i) (void)mbar_wait(c.bars + (i % p.nbuf), (uint32_t)((i / p.nbuf) & 1));
        }
        __syncthreads();
    }
}

// ||a^ - b^||^2 from <a,a>, <b,b>, <a,b>; a zero vector normalises to zero
__device__ __forceinline__ float dissim_sq_from_dot(float saa, float sbb, float sab) {
    const float ca = fmaxf(sqrtf(saa), kNormEps), cb = fmaxf(sqrtf(sbb), kNormEps);
    return fmaxf(saa / (ca * ca) + sbb / (cb * cb) - 2.f * sab / (ca * cb), 0.f);
}

// One CTA per frame: adds the slices in a fixed order, writes S, T, I, ratio_t and k_t.
template <int DT>
__global__ void __launch_bounds__(kFinThreads)
score_finalize_kernel(const FusedParams p) {
    __shared__ float f_s2[kMaxTokensFused], f_t2[kMaxTokensFused], f_aa[kMaxTokensFused], f_bb[kMaxTokensFused];
    __shared__ int f_fl[kMaxTokensFused];
    __shared__ float red[kFinThreads / 32];
    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool is_first = frame_is_first(p.video_frame_offsets, p.num_videos, t);
    // everything the pass kernel wrote is visible after this point
    cudaGridDependencySynchronize();

    // ||mean||^2, fixed order
    const float* mean = p.mean + (int64_t)t * p.d;
    float sm = 0.f;
    for (int c = tid * 4; c < p.d; c += kFinThreads * 4) {
        const float4 m = __ldcg(reinterpret_cast<const float4*>(mean + c));
        sm = fmaf(m.x, m.x, sm); sm = fmaf(m.y, m.y, sm); sm = fmaf(m.z, m.z, sm); sm = fmaf(m.w, m.w, sm);
    }
    sm = warp_sum(sm);
    if (lane == 0) red[warp] = sm;
    __syncthreads();
    float smm = 0.f;
#pragma unroll
    for (int i = 0; i < kFinThreads / 32; ++i) smm += red[i];
    __syncthreads();

    if (tid < p.f) {
        float aa = 0.f, db = 0.f, bb = 0.f, am = 0.f;
        const float4* src = p.part + ((int64_t)t * p.nsl) * p.f + tid;
        int s = 0;
        for (; s + 4 <= p.nsl; s += 4) {
            float4 q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) q[i] = __ldcg(src + (int64_t)(s + i) * p.f);
#pragma unroll
            for (int i = 0; i < 4; ++i) { aa += q[i].x; db += q[i].y; bb += q[i].z; am += q[i].w; }
        }
        for (; s < p.nsl; ++s) {
            const float4 q = __ldcg(src + (int64_t)s * p.f);
            aa += q.x; db += q.y; bb += q.z; am += q.w;
        }
        const float s2 = dissim_sq_from_dot(aa, smm, am);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);
        int fl = 0;
        if (s2 < kRefineBelow) fl |= 1;
        if (!is_first && t2 < kRefineBelow && db != 0.f) fl |= 2;
        f_s2[tid] = s2; f_t2[tid] = t2; f_aa[tid] = aa; f_bb[tid] = bb; f_fl[tid] = fl;
    }
    __syncthreads();
    // nearly parallel rows: exact re-evaluation from the rows themselves (rare)
    for (int row = warp; row < p.f; row += kFinThreads / 32) {
        const int fl = f_fl[row];
        if (fl) {
            const char* pa = p.tokens + ((int64_t)t * p.f + row) * p.row_bytes_ld;
            const char* pb = pa - (int64_t)p.f * p.row_bytes_ld;
            const float ia = 1.f / fmaxf(sqrtf(f_aa[row]), kNormEps);
            const float ib = 1.f / fmaxf(sqrtf(f_bb[row]), kNormEps);
            const float im = 1.f / fmaxf(sqrtf(smm), kNormEps);
            float es, et;
            refine_row<DT>(pa, pb, mean, p.nvec, lane, (fl & 1) != 0, (fl & 2) != 0, ia, ib, im, es, et);
            if (lane == 0) {
                if (fl & 1) f_s2[row] = es;
                if (fl & 2) f_t2[row] = et;
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
    if (lane == 0) red[warp] = tsq;
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

size_t fixed_smem_bytes(int se) { return (size_t)(kRowGroups * se + 4 * se + se) * 4 + 4 * 8 + 16; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            ptr = nullptr;
        }
        return (EncodeTiledFn)ptr;
    }();
    return fn;
}

template <int DT>
sharpv_status launch(const FusedScoreArgs& a, const CUtensorMap& tmap, FusedParams& p, int sms) {
    const size_t fixed = fixed_smem_bytes(Pass<DT>::SE);
    p.nbuf = 3;
    while (p.nbuf > 1 && (size_t)p.nbuf * p.tile_stride + fixed > (size_t)kSmemBudget) --p.nbuf;
    const size_t smem = (size_t)p.nbuf * p.tile_stride + fixed;
    if (smem > (size_t)kSmemBudget) return SHARPV_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(score_pass_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_UNSUPPORTED;
    }
    const int64_t units = (int64_t)p.nsl * a.F;
    const unsigned grid = (unsigned)(units < sms ? units : sms);
    score_pass_kernel<DT><<<grid, kThreads, smem, a.stream>>>(tmap, p, a.status_word);
    if (cudaGetLastError() != cudaSuccess) return SHARPV_ERR_CUDA;

    // the finaliser starts while the pass drains and waits for it with cudaGridDependencySynchronize
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.F);
    cfg.blockDim = dim3(kFinThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, score_finalize_kernel<DT>, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }
    return SHARPV_OK;
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
    EncodeTiledFn enc = encode_fn();
    if (!enc) return SHARPV_ERR_UNSUPPORTED;
    const int eb = elem_bytes(a.dtype);
    FusedParams p;
    p.tokens = (const char*)a.tokens;
    p.row_bytes_ld = a.ld_tokens * eb;
    p.F = a.F; p.f = a.f; p.d = a.d;
    p.nsl = (int)((int64_t)a.d * eb / kSliceBytes);
    p.nvec = a.d * eb / 16;
    p.nbuf = 3;
    p.num_videos = a.num_videos;
    p.video_frame_offsets = a.video_frame_offsets;
    p.w = a.w; p.one_minus_cos = a.one_minus_cos; p.round_mode = a.round_mode; p.min_keep = a.min_keep;
    p.out_I = a.out_I; p.out_S = a.out_S; p.out_T = a.out_T; p.out_ratio = a.out_ratio; p.out_k = a.out_k;
    char* w = (char*)a.workspace;
    p.mean = (float*)w;       w += align_up((size_t)a.F * a.d * 4, 256);
    p.part = (float4*)w;
    p.tile_bytes = (uint32_t)a.f * kSliceBytes;
    p.tile_stride = (uint32_t)align_up((size_t)p.tile_bytes, 128);

    // the token matrix as a byte tensor [rows, d * elem_bytes]; one box is one (frame, slice) tile
    CUtensorMap tmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)a.d * eb, (cuuint64_t)a.F * a.f};
    const cuuint64_t gstr[1] = {(cuuint64_t)p.row_bytes_ld};
    const cuuint32_t box[2] = {(cuuint32_t)kSliceBytes, (cuuint32_t)a.f};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)a.tokens, gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SHARPV_ERR_UNSUPPORTED;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return SHARPV_ERR_CUDA;
    return a.dtype == SHARPV_F32 ? launch<SHARPV_F32>(a, tmap, p, sms) : launch<SHARPV_BF16>(a, tmap, p, sms);
}

}  // namespace sharpv
