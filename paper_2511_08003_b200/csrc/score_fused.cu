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
constexpr int kRowGroups = kThreads / 8;
constexpr int kRows = 4;                // row slots per thread: frames of up to 256 tokens
constexpr int kMaxTokensFused = 256;
constexpr int kSmemBudget = 227 * 1024;
constexpr uint32_t kSpinLimit = 1u << 22;      // polls of one mbarrier before a wait gives up
constexpr int kFinThreads = 1024;

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
// one 32-bit word of two bf16 -> the two exact fp32 values (a bf16 is the upper half of an fp32):
// one multiply and one mask, on different pipes, written straight into the halves of the result
__device__ __forceinline__ f32x2 widen_bf16x2(uint32_t w) {
    f32x2 r;
    asm("{\n\t.reg .b32 lo, hi;\n\t"
        "mul.lo.u32 lo, %1, 65536;\n\t"          // low element: shift up (multiply pipe)
        "and.b32 hi, %1, 0xffff0000;\n\t"        // high element: mask (logic pipe)
        "mov.b64 %0, {lo, hi};\n\t}"
        : "=l"(r) : "r"(w));
    return r;
}
__device__ __forceinline__ f32x2 pair_f32(uint32_t lo, uint32_t hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
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
    static constexpr int H = P / 2;                         // packed pairs per vector
    static constexpr int SE = kSliceBytes / E::kBytes;      // elements per slice row

    const CUtensorMap* tmap;
    const FusedParams* p;
    unsigned char* tiles;
    float* cs;              // [kRowGroups][SE] column sums of each row group
    float* cs2;             // [4][SE]
    float* mean_s;          // [SE]
    uint64_t* bars;         // [nbuf]
    volatile int* abort_flag;
    int Q, halo;
    int load_s, load_t;     // (slice, frame) of the next tile to request (thread 0 only)

    // per-thread state carried from frame to frame
    uint4 prev[kRows][2];   // previous frame's rows of this thread (two vectors each)
    f32x2 mprev[2][H];      // previous frame's mean over this thread's columns
    float bb[kRows];        // this thread's share of ||previous row||^2

    int tid, warp, g, j, rgid;

    // requests tile q; tiles are requested in unit order, so (load_s, load_t) just advances
    __device__ __forceinline__ void issue_load(int q) {
        const FusedParams& pp = *p;
        const int slot = q % pp.nbuf;
        uint64_t* bar = bars + slot;
        mbar_expect_tx(bar, pp.tile_bytes);
        tma_load_2d(tiles + (size_t)slot * pp.tile_stride, tmap, load_s * kSliceBytes, load_t * pp.f, bar);
        if (++load_t == pp.F) { load_t = 0; ++load_s; }
    }

    __device__ __forceinline__ const unsigned char* wait_tile(int slot, uint32_t phase) const {
        if (!mbar_wait(bars + slot, phase)) *abort_flag = 1;
        return tiles + (size_t)slot * p->tile_stride;
    }

    __device__ __forceinline__ static void to_pairs(const uint4& v, f32x2 (&o)[H]) {
        if (DT == SHARPV_BF16) {
            o[0] = widen_bf16x2(v.x); o[1] = widen_bf16x2(v.y);
            o[H - 2] = widen_bf16x2(v.z); o[H - 1] = widen_bf16x2(v.w);
        } else {
            o[0] = pair_f32(v.x, v.y); o[H - 1] = pair_f32(v.z, v.w);
        }
    }

    // Row slot r of this thread is row 64 r + 4 warp + g (g = lane group): a warp owns four
    // consecutive rows per slot.  A slot is visited when its first row exists (a warp-uniform test);
    // lane groups whose row lies beyond the frame read the zero rows that pad every tile buffer to a
    // multiple of four rows, so no lane ever branches on its own row.
    __device__ __forceinline__ bool slot_live(int r) const { return 64 * r + 4 * warp < p->f; }
    __device__ __forceinline__ int slot_row(int r) const { return 64 * r + 4 * warp + g; }
    __device__ __forceinline__ const unsigned char* my_rows(const unsigned char* tile) const {
        return tile + (4 * warp + g) * kSliceBytes + j * 16;
    }

    // Frame in front of the first unit: registers only.
    __device__ __forceinline__ void load_halo(const unsigned char* tile) {
        const unsigned char* base = my_rows(tile);
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            f32x2 acc = pk(0.f, 0.f);
            if (slot_live(r)) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    prev[r][h] = *reinterpret_cast<const uint4*>(base + r * (64 * kSliceBytes) + h * 128);
                    f32x2 b2[H];
                    to_pairs(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc = fma2(b2[i], b2[i], acc);
                }
            }
            bb[r] = hsum(acc);
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
            if (slot_live(r)) {
                f32x2 acc = pk(0.f, 0.f);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    f32x2 b2[H];
                    to_pairs(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc = fma2(b2[i], mprev[h][i], acc);
                }
                x[4 * r + 3] = hsum(acc);
            }
        }
        group8_reduce_scatter(x, j);
        const int row = slot_row(j >> 1);
        if ((j & 1) && row < p->f) p->part[((int64_t)t_prev * p->nsl + s) * p->f + row].w = x[1];
    }

    // Slots [R0, R1) of one tile, without a branch: everything the frame contributes per row.
    //   HAS_PREV  the registers hold frame t-1 of this slice
    //   TEMPORAL  ... and frame t continues the same video, so ||a-b||^2 is wanted
    //   OWN_PREV  ... and frame t-1 was a unit of this CTA, so its <row, mean> is computed here
    template <int R0, int R1, bool HAS_PREV, bool TEMPORAL, bool OWN_PREV>
    __device__ __forceinline__ void slots(const unsigned char* base, f32x2 (&colsum)[2][H], float (&x)[16]) {
        uint4 a4[R1 - R0][2];
#pragma unroll
        for (int r = R0; r < R1; ++r)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                a4[r - R0][h] = *reinterpret_cast<const uint4*>(base + r * (64 * kSliceBytes) + h * 128);
#pragma unroll
        for (int r = R0; r < R1; ++r) {
            f32x2 aa = pk(0.f, 0.f), db = aa, bm = aa;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                f32x2 a2[H];
                to_pairs(a4[r - R0][h], a2);
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    colsum[h][i] = add2(colsum[h][i], a2[i]);
                    aa = fma2(a2[i], a2[i], aa);
                }
                if (HAS_PREV && (TEMPORAL || OWN_PREV)) {
                    f32x2 b2[H];
                    to_pairs(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) {
                        if (TEMPORAL) {
                            const f32x2 e = sub2(a2[i], b2[i]);
                            db = fma2(e, e, db);
                        }
                        if (OWN_PREV) bm = fma2(b2[i], mprev[h][i], bm);
                    }
                }
                prev[r][h] = a4[r - R0][h];
            }
            x[4 * r + 0] = hsum(aa);
            x[4 * r + 1] = hsum(db);
            x[4 * r + 2] = HAS_PREV ? bb[r] : 0.f;
            x[4 * r + 3] = hsum(bm);
            bb[r] = x[4 * r + 0];
        }
    }

    // One unit: the tile of (slice s, frame t) in buffer `slot`; q is its place in the load order.
    // Returns false when the CTA must stop (a bounded wait ran out).
    template <bool HAS_PREV, bool TEMPORAL, bool OWN_PREV>
    __device__ __forceinline__ bool unit(int q, int slot, uint32_t phase, int s, int t) {
        const FusedParams& pp = *p;
        const unsigned char* base = my_rows(wait_tile(slot, phase));

        f32x2 colsum[2][H];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < H; ++i) colsum[h][i] = pk(0.f, 0.f);
        float x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = 0.f;
        if (slot_live(2)) {                     // the usual case: a straight run over three slots
            slots<0, 2, HAS_PREV, TEMPORAL, OWN_PREV>(base, colsum, x);
            slots<2, 3, HAS_PREV, TEMPORAL, OWN_PREV>(base, colsum, x);
            if (slot_live(3)) slots<3, 4, HAS_PREV, TEMPORAL, OWN_PREV>(base, colsum, x);
        } else {
            if (slot_live(0)) slots<0, 1, HAS_PREV, TEMPORAL, OWN_PREV>(base, colsum, x);
            if (slot_live(1)) slots<1, 2, HAS_PREV, TEMPORAL, OWN_PREV>(base, colsum, x);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float* dst = cs + rgid * SE + (j + 8 * h) * P;
#pragma unroll
            for (int i = 0; i < H; i += 2)
                *reinterpret_cast<ulonglong2*>(dst + 2 * i) = make_ulonglong2(colsum[h][i], colsum[h][i + 1]);
        }
        __syncthreads();                            // tile buffer free, column partials visible
        if (*abort_flag) return false;
        if (tid == 0 && q + pp.nbuf < Q) issue_load(q + pp.nbuf);
        // column sums over the 64 row groups: fixed order, two levels
#pragma unroll
        for (int e = tid; e < 4 * SE; e += kThreads) {
            const int col = e % SE, quarter = e / SE;
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < kRowGroups / 4; ++i) sum += cs[(quarter * (kRowGroups / 4) + i) * SE + col];
            cs2[quarter * SE + col] = sum;
        }

        // per-row partial sums of the slice (overlaps the mean reduction of the other warps)
        group8_reduce_scatter(x, j);
        {
            const int row = slot_row(j >> 1);
            if (row < pp.f) {
                float4* rec = pp.part + ((int64_t)t * pp.nsl + s) * pp.f + row;
                if (j & 1) {
                    rec->z = x[0];                                              // ||b||^2
                    if (OWN_PREV) (rec - (int64_t)pp.nsl * pp.f)->w = x[1];     // frame t-1: <b, mean>
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
                mprev[h][i] = *reinterpret_cast<const f32x2*>(mean_s + (j + 8 * h) * P + 2 * i);
        return true;
    }

    __device__ __forceinline__ bool unit_dispatch(int q, int slot, uint32_t phase, int s, int t, bool has_prev,
                                                  bool own_prev, bool is_first) {
        if (!has_prev) return unit<false, false, false>(q, slot, phase, s, t);
        if (!is_first)
            return own_prev ? unit<true, true, true>(q, slot, phase, s, t)
                            : unit<true, true, false>(q, slot, phase, s, t);
        return own_prev ? unit<true, false, true>(q, slot, phase, s, t)
                        : unit<true, false, false>(q, slot, phase, s, t);
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

    // let the finaliser's CTAs be scheduled as soon as SMs free up; they wait for this whole grid
    cudaTriggerProgrammaticLaunchCompletion();
    cudaGridDependencySynchronize();        // the tokens come from earlier work on the stream
    const int64_t U = (int64_t)p.nsl * p.F;
    const int64_t u0 = U * blockIdx.x / gridDim.x;
    const int64_t u1 = U * (blockIdx.x + 1) / gridDim.x;
    if (u0 >= u1) return;
    int s = (int)(u0 / p.F), t = (int)(u0 % p.F);

    // videos: `vid` is the video of frame t, `next_start` the first frame of the next one
    int vid = upper_segment(p.video_frame_offsets, p.num_videos, t);
    bool is_first = __ldg(p.video_frame_offsets + vid) == t;
    int next_start = __ldg(p.video_frame_offsets + vid + 1);

    c.halo = is_first ? 0 : 1;
    c.Q = (int)(u1 - u0) + c.halo;
    c.load_s = s;
    c.load_t = t - c.halo;

    const int tid = threadIdx.x, lane = tid & 31;
    c.tid = tid;
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
    // rows beyond the frame in every tile buffer stay zero for the whole kernel (TMA writes f rows)
    for (int b = 0; b < p.nbuf; ++b) {
        uint4* pad = reinterpret_cast<uint4*>(c.tiles + (size_t)b * p.tile_stride + p.tile_bytes);
        const int n = (int)((p.tile_stride - p.tile_bytes) / 16);
        for (int i = tid; i < n; i += kThreads) pad[i] = make_uint4(0u, 0u, 0u, 0u);
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

    int q = 0, slot = 0;
    uint32_t phase = 0;
    bool ok = true, has_prev = false, own_prev = false;
    if (c.halo) {
        c.load_halo(c.wait_tile(0, 0));
        __syncthreads();
        ok = *c.abort_flag == 0;
        if (ok && tid == 0 && p.nbuf < c.Q) c.issue_load(p.nbuf);
        q = 1;
        if (++slot == p.nbuf) { slot = 0; phase ^= 1; }
        has_prev = true;
    }
    const int n_units = (int)(u1 - u0);
    for (int i = 0; ok && i < n_units; ++i) {
        ok = c.unit_dispatch(q, slot, phase, s, t, has_prev, own_prev, is_first);
        has_prev = true;
        own_prev = true;
        ++q;
        if (++slot == p.nbuf) { slot = 0; phase ^= 1; }
        // next unit
        if (++t == p.F) {                           // the range crosses into the next slice
            if (ok) c.flush_prev(s, p.F - 1);
            t = 0;
            ++s;
            has_prev = false;
            own_prev = false;
            vid = upper_segment(p.video_frame_offsets, p.num_videos, 0);
            next_start = __ldg(p.video_frame_offsets + vid + 1);
            is_first = true;
        } else {
            is_first = false;
            while (t >= next_start && vid + 1 < p.num_videos) {     // skips videos without frames
                ++vid;
                is_first = true;
                next_start = __ldg(p.video_frame_offsets + vid + 1);
            }
        }
    }
    if (ok) {
        if (own_prev) c.flush_prev((int)((u1 - 1) / p.F), (int)((u1 - 1) % p.F));
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
        const float aa = (a0.x + a1.x) + (a2.x + a3.x), db = (a0.y + a1.y) + (a2.y + a3.y);
        const float bb = (a0.z + a1.z) + (a2.z + a3.z), am = (a0.w + a1.w) + (a2.w + a3.w);
        const float s2 = dissim_sq_from_dot(aa, smm, am);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);
        int fl = 0;
        if (s2 < kRefineBelow) fl |= 1;
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
    if (launch_dependent(score_pass_kernel<DT>, dim3(grid), dim3(kThreads), smem, a.stream, tmap, p,
                         a.status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_CUDA;
    }

    // the finaliser starts while the pass drains and waits for it with cudaGridDependencySynchronize
    if (launch_dependent(score_finalize_kernel<DT>, dim3((unsigned)a.F), dim3(kFinThreads), 0, a.stream, p) !=
        cudaSuccess) {
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
    p.tile_stride = (uint32_t)((a.f + 3) / 4 * 4) * kSliceBytes;   // whole groups of four rows; the tail stays zero

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
