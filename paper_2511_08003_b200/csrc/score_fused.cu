// Stage one (a) with one HBM read per token (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// The token matrix is cut into column slices of 256 bytes.  A work unit is (slice s, frame t):
// the f x 256-byte tile of frame t.  Persistent CTAs (one per SM) each take a contiguous range of
// units in (slice-major, frame-minor) order, so a CTA walks consecutive frames of one slice.
//
//   score_pass_kernel      640 threads in two roles that only meet through mbarriers:
//       column warps (4)   issue the TMA loads that fill a ring of tile buffers, add up the columns
//                          of each tile (the whole frame column is inside the tile, so this is the
//                          slice of the frame mean) and publish the mean one tile ahead of the rows;
//       row warps (16)     keep their part of the previous frame's tile in registers (4 rows x two
//                          16-byte vectors per thread), visit each new tile once for ||a||^2,
//                          ||a - mean||^2 and ||a - b||^2 with packed fp32 FMAs, overwrite the old
//                          rows in place and write one record of partial sums per row and slice.
//       Every wait is on the CTA's own barriers and is bounded.
//   score_finalize_kernel  one CTA per frame, launched as a programmatic dependent so that its
//       start-up overlaps the tail of the pass: adds the slices in a fixed order and writes
//       S, T, I, the ratio and the budget of the frame.
#include <cuda.h>

#include "score_common.cuh"
#include "score_fused.cuh"

namespace sharpv {
namespace {

constexpr int kSliceBytes = 256;
constexpr int kRowWarps = 16;           // a row warp = 4 row groups x 8 lanes (two vectors per lane)
constexpr int kColWarps = 4;            // 128 threads = 16 vector columns x 8 row groups
constexpr int kRowThreads = kRowWarps * 32;
constexpr int kColThreads = kColWarps * 32;
constexpr int kThreads = kRowThreads + kColThreads;
constexpr int kColGroups = kColThreads / 16;
constexpr int kRows = 4;                // row slots per row-warp thread: frames of up to 256 tokens
constexpr int kMaxTokensFused = 256;
constexpr int kNBuf = 3;                // tile buffers in the ring
constexpr int kSmemBudget = 227 * 1024;
constexpr uint32_t kSpinLimit = 1u << 24;      // polls of one mbarrier before a wait gives up
constexpr long long kSpinClocks = 2000000000ll; // ... or about one second of SM clock
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
    float4* part;           // [F, nsl, f]: (||a||^2, ||a-m||^2, ||a-b||^2, ||b||^2) of the slice
    uint32_t tile_bytes, tile_stride;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// bounded wait: false when the limit ran out (a poll count and, every 256 polls, about a second of
// SM clock, whichever comes first)
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 0 && clock64() - t0 > kSpinClocks) return false;
    }
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

// Shared-memory layout of one CTA.
template <int DT>
struct Smem {
    static constexpr int SE = kSliceBytes / Elem<DT>::kBytes;       // elements per slice row
    unsigned char* tiles;       // [kNBuf][tile_stride]
    float* cs;                  // [kColGroups][SE] column sums of each row group of the column warps
    float* mean_s;              // [2][SE] frame-mean slice of the tiles, alternating
    uint64_t* full;             // [kNBuf] tile landed (TMA)
    uint64_t* empty;            // [kNBuf] tile released by all 20 warps
    uint64_t* mean_full;        // [2] mean published by the column warps
    uint64_t* mean_empty;       // [2] mean read by all 16 row warps
    volatile int* abort_flag;

    __device__ __forceinline__ Smem(unsigned char* base, uint32_t tile_stride) {
        tiles = base;
        cs = reinterpret_cast<float*>(base + (size_t)kNBuf * tile_stride);
        mean_s = cs + kColGroups * SE;
        full = reinterpret_cast<uint64_t*>(mean_s + 2 * SE);
        empty = full + kNBuf;
        mean_full = empty + kNBuf;
        mean_empty = mean_full + 2;
        abort_flag = reinterpret_cast<volatile int*>(mean_empty + 2);
    }
    static size_t fixed_bytes() { return (size_t)(kColGroups * SE + 2 * SE) * 4 + (2 * kNBuf + 4) * 8 + 16; }
};

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

// barrier 1 over the column warps with an OR of `flag`: every thread gets the same answer
__device__ __forceinline__ bool column_any(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out) : "r"((uint32_t)flag), "n"(kColThreads) : "memory");
    return out != 0;
}

// ---------------------------------------------------------------------------------------
// column warps: TMA producer, column sums, frame mean
// ---------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void column_role(const CUtensorMap* tmap, const FusedParams& p, Smem<DT>& sm, int64_t u0,
                                            int n_units, int halo, int ctid) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec, H = P / 2, SE = Smem<DT>::SE;
    const int Q = n_units + halo;
    const int vcol = ctid & 15, rgrp = ctid >> 4, lane = ctid & 31;

    // tiles are requested in unit order: (load_s, load_t) just advances (thread 0 of the role)
    int load_s = (int)(u0 / p.F), load_t = (int)(u0 % p.F) - halo;
    auto issue = [&](int slot) {
        mbar_expect_tx(sm.full + slot, p.tile_bytes);
        tma_load_2d(sm.tiles + (size_t)slot * p.tile_stride, tmap, load_s * kSliceBytes, load_t * p.f,
                    sm.full + slot);
        if (++load_t == p.F) { load_t = 0; ++load_s; }
    };
    if (ctid == 0)
        for (int q = 0; q < kNBuf && q < Q; ++q) issue(q);

    Walk w;
    w.start(p, u0);
    // ring position of tile q and of tile q-1, and the mean buffer of unit n, all kept incrementally
    int slot = 0, prev_slot = 0, mb = 0;
    uint32_t phase = 0, prev_phase = 0, mean_empty_phase = 1;
    float* mean_out = p.mean + (int64_t)w.t * p.d + w.s * SE + ctid;
    for (int q = 0; q < Q; ++q) {
        const bool halo_tile = halo && q == 0;
        // the 128 threads leave together: a thread that saw a failed wait tells the others here
        bool bad = *sm.abort_flag != 0;
        if (!bad && !halo_tile && !mbar_wait(sm.full + slot, phase)) {
            *sm.abort_flag = 1;
            bad = true;
        }
        if (column_any(bad)) return;
        if (halo_tile) {
            if (lane == 0) mbar_arrive(sm.empty + slot);        // the column warps do not read the halo tile
        } else {
            const int n = q - halo;
            const unsigned char* tile = sm.tiles + (size_t)slot * p.tile_stride + vcol * 16;
            f32x2 acc[H];
#pragma unroll
            for (int i = 0; i < H; ++i) acc[i] = pk(0.f, 0.f);
            int r = rgrp;
            for (; r + 3 * kColGroups < p.f; r += 4 * kColGroups) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    v[u] = *reinterpret_cast<const uint4*>(tile + (r + u * kColGroups) * kSliceBytes);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    f32x2 a2[H];
                    widen_pairs<DT>(v[u], a2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc[i] = add2(acc[i], a2[i]);
                }
            }
            for (; r < p.f; r += kColGroups) {
                f32x2 a2[H];
                widen_pairs<DT>(*reinterpret_cast<const uint4*>(tile + r * kSliceBytes), a2);
#pragma unroll
                for (int i = 0; i < H; ++i) acc[i] = add2(acc[i], a2[i]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.empty + slot);        // this warp is done with the tile
            float* dst = sm.cs + rgrp * SE + vcol * P;
#pragma unroll
            for (int i = 0; i < H; i += 2)
                *reinterpret_cast<ulonglong2*>(dst + 2 * i) = make_ulonglong2(acc[i], acc[i + 1]);
            asm volatile("bar.sync 1, %0;" ::"n"(kColThreads) : "memory");
            if (ctid < SE) {
                float sum = 0.f;
#pragma unroll
                for (int gidx = 0; gidx < kColGroups; ++gidx) sum += sm.cs[gidx * SE + ctid];
                const float m = sum / (float)p.f;
                // the buffer was last used two tiles ago: wait until every row warp has read it
                if (n >= 2 && !mbar_wait(sm.mean_empty + mb, mean_empty_phase)) *sm.abort_flag = 1;
                sm.mean_s[mb * SE + ctid] = m;
                *mean_out = m;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kColThreads) : "memory");
            if (ctid == 0) mbar_arrive(sm.mean_full + mb);
            if (mb) mean_empty_phase ^= 1;              // units n and n+1 share a phase of their buffers
            mb ^= 1;
            if (w.step(p)) mean_out = p.mean + w.s * SE + ctid;
            else mean_out += p.d;
        }
        // refill the buffer of the tile in front of this one as soon as every warp has let go of it
        if (ctid == 0 && q >= 1 && q - 1 + kNBuf < Q) {
            if (mbar_wait(sm.empty + prev_slot, prev_phase)) issue(prev_slot);
            else *sm.abort_flag = 1;                            // everyone leaves at the next check
        }
        prev_slot = slot;
        prev_phase = phase;
        if (++slot == kNBuf) { slot = 0; phase ^= 1; }
    }
}

// ---------------------------------------------------------------------------------------
// row warps
// ---------------------------------------------------------------------------------------
template <int DT>
struct RowState {
    static constexpr int H = Elem<DT>::kPerVec / 2;
    uint4 prev[kRows][2];   // previous frame's rows of this thread (two vectors each)
    float bb[kRows];        // this thread's share of ||previous row||^2
    int warp, g, j, f;

    // Row slot r of this thread is row 64 r + 4 warp + g (g = lane group): a warp owns four
    // consecutive rows per slot.  A slot is visited when its first row exists (a warp-uniform test);
    // lane groups whose row lies beyond the frame read the zero rows that pad every tile buffer to a
    // multiple of four rows, so no lane ever branches on its own row.
    __device__ __forceinline__ bool slot_live(int r) const { return 64 * r + 4 * warp < f; }
    __device__ __forceinline__ int slot_row(int r) const { return 64 * r + 4 * warp + g; }
    __device__ __forceinline__ const unsigned char* my_rows(const unsigned char* tile) const {
        return tile + (4 * warp + g) * kSliceBytes + j * 16;
    }

    // frame in front of the first unit: registers only
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
                    widen_pairs<DT>(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) acc = fma2(b2[i], b2[i], acc);
                }
            }
            bb[r] = hsum(acc);
        }
    }

    // slots [R0, R1) of one tile, without a branch: ||a||^2, ||a - m||^2 and, when the frame continues
    // a video (TEMPORAL), ||a - b||^2 against the rows in registers, which the new rows then replace
    template <int R0, int R1, bool TEMPORAL>
    __device__ __forceinline__ void slots(const unsigned char* base, const f32x2 (&m)[2][H], float (&x)[16]) {
        uint4 a4[R1 - R0][2];
#pragma unroll
        for (int r = R0; r < R1; ++r)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                a4[r - R0][h] = *reinterpret_cast<const uint4*>(base + r * (64 * kSliceBytes) + h * 128);
#pragma unroll
        for (int r = R0; r < R1; ++r) {
            f32x2 aa = pk(0.f, 0.f), dm = aa, db = aa;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                f32x2 a2[H];
                widen_pairs<DT>(a4[r - R0][h], a2);
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    const f32x2 e = sub2(a2[i], m[h][i]);
                    aa = fma2(a2[i], a2[i], aa);
                    dm = fma2(e, e, dm);
                }
                if (TEMPORAL) {
                    f32x2 b2[H];
                    widen_pairs<DT>(prev[r][h], b2);
#pragma unroll
                    for (int i = 0; i < H; ++i) {
                        const f32x2 e = sub2(a2[i], b2[i]);
                        db = fma2(e, e, db);
                    }
                }
                prev[r][h] = a4[r - R0][h];
            }
            x[4 * r + 0] = hsum(aa);
            x[4 * r + 1] = hsum(dm);
            x[4 * r + 2] = hsum(db);
            x[4 * r + 3] = TEMPORAL ? bb[r] : 0.f;
            bb[r] = x[4 * r + 0];
        }
    }

    template <bool TEMPORAL>
    __device__ __forceinline__ void tile_pass(const unsigned char* tile, const f32x2 (&m)[2][H], float (&x)[16]) {
        const unsigned char* base = my_rows(tile);
        if (slot_live(2)) {                     // the usual case: a straight run over three slots
            slots<0, 2, TEMPORAL>(base, m, x);
            slots<2, 3, TEMPORAL>(base, m, x);
            if (slot_live(3)) slots<3, 4, TEMPORAL>(base, m, x);
        } else {
            if (slot_live(0)) slots<0, 1, TEMPORAL>(base, m, x);
            if (slot_live(1)) slots<1, 2, TEMPORAL>(base, m, x);
        }
    }
};

template <int DT>
__device__ __forceinline__ void row_role(const FusedParams& p, Smem<DT>& sm, int64_t u0, int n_units, int halo,
                                         int tid) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec, H = P / 2, SE = Smem<DT>::SE;
    const int lane = tid & 31;
    RowState<DT> st;
    st.warp = tid >> 5;
    st.g = lane >> 3;
    st.j = lane & 7;
    st.f = p.f;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        st.prev[r][0] = make_uint4(0u, 0u, 0u, 0u);
        st.prev[r][1] = st.prev[r][0];
        st.bb[r] = 0.f;
    }
    int q = 0;
    bool has_prev = false;
    if (halo) {
        if (!__all_sync(0xffffffffu, mbar_wait(sm.full + 0, 0))) { *sm.abort_flag = 1; return; }
        st.load_halo(sm.tiles);
        __syncwarp();
        if (lane == 0) mbar_arrive(sm.empty + 0);
        q = 1;
        has_prev = true;
    }
    static_assert(kNBuf >= 2, "the halo tile and the first unit need their own buffers");
    Walk w;
    w.start(p, u0);
    // ring position of the tile, mean buffer of the unit and the unit's record block, kept incrementally
    int slot = q, mb = 0;
    uint32_t phase = 0, mean_phase = 0;
    const unsigned char* tile = sm.tiles + (size_t)slot * p.tile_stride;
    const int64_t rec_step = (int64_t)p.nsl * p.f;
    float4* rec_block = p.part + ((int64_t)w.t * p.nsl + w.s) * p.f;
    for (int n = 0; n < n_units; ++n) {
        // a warp leaves as a whole: the lanes agree on what they saw
        const bool fine = *sm.abort_flag == 0 && mbar_wait(sm.full + slot, phase) &&
                          mbar_wait(sm.mean_full + mb, mean_phase);
        if (!__all_sync(0xffffffffu, fine)) {
            *sm.abort_flag = 1;
            return;
        }
        f32x2 m[2][H];
        const float* ms = sm.mean_s + mb * SE;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < H; ++i)
                m[h][i] = *reinterpret_cast<const f32x2*>(ms + (st.j + 8 * h) * P + 2 * i);
        __syncwarp();
        if (lane == 0) mbar_arrive(sm.mean_empty + mb);

        float x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = 0.f;
        if (has_prev && !w.is_first) st.template tile_pass<true>(tile, m, x);
        else st.template tile_pass<false>(tile, m, x);
        __syncwarp();
        if (lane == 0) mbar_arrive(sm.empty + slot);            // this warp is done with the tile

        // per-row sums of the slice: reduce over the row's 8 lanes, one record per row
        group8_reduce_scatter(x, st.j);
        const int row = st.slot_row(st.j >> 1);
        if (row < p.f)      // even lane: ||a||^2, ||a-m||^2; odd lane: ||a-b||^2, ||b||^2
            reinterpret_cast<float2*>(rec_block + row)[st.j & 1] = make_float2(x[0], x[1]);
        if (w.step(p)) {                                // a new slice starts without a previous frame
            has_prev = false;
            rec_block = p.part + (int64_t)w.s * p.f;
        } else {
            has_prev = true;
            rec_block += rec_step;
        }
        if (mb) mean_phase ^= 1;
        mb ^= 1;
        tile += p.tile_stride;
        if (++slot == kNBuf) { slot = 0; phase ^= 1; tile = sm.tiles; }
    }
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
score_pass_kernel(const __grid_constant__ CUtensorMap tmap, const FusedParams p, int32_t* status_word) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Smem<DT> sm(smem, p.tile_stride);

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

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int i = 0; i < kNBuf; ++i) {
            mbar_init(sm.full + i, 1);
            mbar_init(sm.empty + i, kRowWarps + kColWarps);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(sm.mean_full + i, 1);
            mbar_init(sm.mean_empty + i, kRowWarps);
        }
        *sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // rows beyond the frame in every tile buffer stay zero for the whole kernel (TMA writes f rows)
    for (int b = 0; b < kNBuf; ++b) {
        uint4* pad = reinterpret_cast<uint4*>(sm.tiles + (size_t)b * p.tile_stride + p.tile_bytes);
        const int n = (int)((p.tile_stride - p.tile_bytes) / 16);
        for (int i = tid; i < n; i += kThreads) pad[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();

    // The block is launched with 96 registers per thread (640 x 96 = 61440).  The column warps give
    // most of theirs back and the four row warpgroups take 8 more each: 128 x 48 + 512 x 104 = 59392.
    if (tid < kRowThreads) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
        row_role<DT>(p, sm, u0, n_units, halo, tid);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        column_role<DT>(&tmap, p, sm, u0, n_units, halo, tid - kRowThreads);
    }

    __syncthreads();
    if (*sm.abort_flag && tid == 0) {
        // A bounded wait ran out.  Report it, then give every tile buffer one more bounded wait so
        // that no load lands in shared memory after the CTA has gone.
        report(status_word, SHARPV_ERR_TIMEOUT);
        for (int i = 0; i < kNBuf; ++i) {
            (void)mbar_wait(sm.full + i, 0);
            (void)mbar_wait(sm.full + i, 1);
        }
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
        const float aa = (a0.x + a1.x) + (a2.x + a3.x), dm = (a0.y + a1.y) + (a2.y + a3.y);
        const float db = (a0.z + a1.z) + (a2.z + a3.z), bb = (a0.w + a1.w) + (a2.w + a3.w);
        const float s2 = dissim_sq_from_sums(aa, smm, dm);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);
        int fl = 0;
        if (s2 < kRefineBelow && dm != 0.f) fl |= 1;
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
    const size_t smem = (size_t)kNBuf * p.tile_stride + Smem<DT>::fixed_bytes();
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
