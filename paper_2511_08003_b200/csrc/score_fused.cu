// Stage one (a) in a single kernel (Section 3.1.2 - 3.1.3, Eq. 1-6): every token is read from
// HBM once.
//
// The token matrix is cut into column slices of 256 bytes.  A work unit is (slice c, frame t):
// the f x 256-byte tile of frame t.  Persistent CTAs (one per SM) each take a contiguous range of
// units in (slice-major, frame-minor) order, so a CTA walks consecutive frames of one slice:
//   - TMA brings the next tiles into a ring of shared-memory buffers while the current one is
//     being reduced;
//   - each thread copies its part of the tile into registers (13 rows x one 16-byte vector) and
//     keeps the previous frame's copy, so the temporal term needs no second read;
//   - the column sums of the tile give the slice of the frame mean (the whole frame column is
//     inside the tile), after which the per-row sums ||a||^2, ||a-m||^2, ||a-b||^2, ||b||^2 follow
//     from registers with packed fp32 FMAs;
//   - the per-row partial sums of the slice go to a small workspace; the CTA that completes a
//     frame's last slice (an integer ticket per frame) adds the slices in a fixed order and
//     writes S, T, I, the ratio and the budget of that frame.
// Nothing waits on another CTA; the only wait is on the CTA's own TMA loads and it is bounded.
#include <cuda.h>

#include "score_common.cuh"
#include "score_fused.cuh"

namespace sharpv {
namespace {

constexpr int kSliceBytes = 256;
constexpr int kThreads = 256;           // 16 row groups x 16 vectors
constexpr int kRowGroups = 16;
constexpr int kRMax = 13;               // rows per thread: frames of up to 208 tokens
constexpr int kMaxTokensFused = kRowGroups * kRMax;
constexpr int kNBuf = 3;                // tile buffers in flight
constexpr uint32_t kSpinLimit = 1u << 22;  // polls of one mbarrier before a wait gives up

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
    float* part;            // [F, nsl, f, 4]: ||a||^2, ||a-m||^2, ||a-b||^2, ||b||^2 per slice
    int32_t* counters;      // [F] slices completed
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

__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

// 16 lanes x 64 values -> lane L of the group ends with the 4 values of slot L (values are laid
// out slot-major, x[4*slot + j]).  Fixed pairing, hence a fixed summation order.
__device__ __forceinline__ void group16_reduce_scatter(float (&x)[64], int lane16) {
    {
        const bool up = lane16 & 8;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float lo = x[i], hi = x[32 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 8);
        }
    }
    {
        const bool up = lane16 & 4;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float lo = x[i], hi = x[16 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 4);
        }
    }
    {
        const bool up = lane16 & 2;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float lo = x[i], hi = x[8 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 2);
        }
    }
    {
        const bool up = lane16 & 1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = x[i], hi = x[4 + i];
            x[i] = (up ? hi : lo) + __shfl_xor_sync(0xffffffffu, up ? lo : hi, 1);
        }
    }
}

template <int DT>
struct Ctx {
    using E = Elem<DT>;
    static constexpr int P = E::kPerVec;
    static constexpr int SE = kSliceBytes / E::kBytes;      // elements per slice row
    const CUtensorMap* tmap;
    const FusedParams* p;
    unsigned char* tiles;
    float* cs;              // [16][SE] column-sum partials
    float* mean_s;          // [SE]
    float* fin;             // [6][kMaxTokensFused] finaliser scratch
    uint64_t* bars;         // [kNBuf]
    volatile int* flags;    // [0] abort, [1] last-slice ticket
    int64_t u0;
    int Q, halo;
};

__device__ __forceinline__ bool frame_is_first(const FusedParams& p, int t) {
    const int b = upper_segment(p.video_frame_offsets, p.num_videos, t);
    return __ldg(p.video_frame_offsets + b) == t;
}

template <int DT>
__device__ __forceinline__ void issue_load(const Ctx<DT>& c, int q) {
    const FusedParams& p = *c.p;
    int64_t u = c.u0 + q - c.halo;
    int t, s;
    if (c.halo && q == 0) { s = (int)(c.u0 / p.F); t = (int)(c.u0 % p.F) - 1; }
    else { s = (int)(u / p.F); t = (int)(u % p.F); }
    uint64_t* bar = c.bars + (q % kNBuf);
    mbar_expect_tx(bar, p.tile_bytes);
    tma_load_2d(c.tiles + (size_t)(q % kNBuf) * p.tile_stride, c.tmap, s * kSliceBytes, t * p.f, bar);
}

// Copies this thread's part of tile q into registers; returns the column sums of those rows.
template <int DT>
__device__ __forceinline__ void tile_to_regs(const Ctx<DT>& c, int q, int rg, int v, uint4 (&dst)[kRMax],
                                             float (&colsum)[Ctx<DT>::P]) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    if (!mbar_wait(c.bars + (q % kNBuf), (uint32_t)((q / kNBuf) & 1))) c.flags[0] = 1;
    const unsigned char* tile = c.tiles + (size_t)(q % kNBuf) * c.p->tile_stride;
#pragma unroll
    for (int j = 0; j < P; ++j) colsum[j] = 0.f;
#pragma unroll
    for (int r = 0; r < kRMax; ++r) {
        const int row = rg + kRowGroups * r;
        if (row < c.p->f) {
            dst[r] = *reinterpret_cast<const uint4*>(tile + row * kSliceBytes + v * 16);
            float x[P];
            E::widen(dst[r], x);
#pragma unroll
            for (int j = 0; j < P; ++j) colsum[j] += x[j];
        } else {
            dst[r] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

// The CTA that completed the last slice of frame t: adds the slices, writes the frame's outputs.
template <int DT>
__device__ void finalize_frame(const Ctx<DT>& c, int t, bool is_first) {
    const FusedParams& p = *c.p;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* f_s2 = c.fin;
    float* f_t2 = c.fin + kMaxTokensFused;
    float* f_aa = c.fin + 2 * kMaxTokensFused;
    float* f_bb = c.fin + 3 * kMaxTokensFused;
    float* f_fl = c.fin + 4 * kMaxTokensFused;
    float* red = c.fin + 5 * kMaxTokensFused;       // [16] reduction scratch

    // ||mean||^2, fixed order
    const float* mean = p.mean + (int64_t)t * p.d;
    float sm = 0.f;
    for (int j = tid; j < p.d; j += kThreads) {
        const float m = __ldcg(mean + j);
        sm = fmaf(m, m, sm);
    }
    sm = warp_sum(sm);
    if (lane == 0) red[warp] = sm;
    __syncthreads();
    float smm = 0.f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) smm += red[i];
    __syncthreads();

    if (tid < p.f) {
        float aa = 0.f, dm = 0.f, db = 0.f, bb = 0.f;
        const float4* src = reinterpret_cast<const float4*>(p.part) + ((int64_t)t * p.nsl) * p.f + tid;
        for (int s = 0; s < p.nsl; ++s) {
            const float4 q = __ldcg(src + (int64_t)s * p.f);
            aa += q.x; dm += q.y; db += q.z; bb += q.w;
        }
        const float s2 = dissim_sq_from_sums(aa, smm, dm);
        const float t2 = is_first ? 0.f : dissim_sq_from_sums(aa, bb, db);
        int fl = 0;
        if (s2 < kRefineBelow && dm != 0.f) fl |= 1;
        if (!is_first && t2 < kRefineBelow && db != 0.f) fl |= 2;
        f_s2[tid] = s2; f_t2[tid] = t2; f_aa[tid] = aa; f_bb[tid] = bb; f_fl[tid] = __int_as_float(fl);
    }
    __syncthreads();
    // nearly parallel rows: exact re-evaluation from the rows themselves (rare)
    for (int row = warp; row < p.f; row += kThreads / 32) {
        const int fl = __float_as_int(f_fl[row]);
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
        for (int i = 0; i < kThreads / 32; ++i) tot += red[i];
        const float r = ratio_from_sumsq(tot, p.f);
        p.out_ratio[t] = r;
        p.out_k[t] = budget_from_ratio(r, p.f, p.round_mode, p.min_keep);
    }
    __syncthreads();
}

// One unit: tile q = (slice s, frame t).  `cur` receives the tile, `prev` holds frame t-1.
// Returns false when the CTA must stop (a bounded wait ran out).
template <int DT>
__device__ __forceinline__ bool process_unit(const Ctx<DT>& c, int q, int s, int t, uint4 (&cur)[kRMax],
                                             const uint4 (&prev)[kRMax]) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    constexpr int SE = Ctx<DT>::SE;
    const FusedParams& p = *c.p;
    const int tid = threadIdx.x, v = tid & 15, rg = tid >> 4;
    const bool is_first = frame_is_first(p, t);

    float colsum[P];
    tile_to_regs<DT>(c, q, rg, v, cur, colsum);
#pragma unroll
    for (int j = 0; j < P; ++j) c.cs[rg * SE + v * P + j] = colsum[j];
    __syncthreads();                                    // tile buffer free, column partials visible
    if (c.flags[0]) return false;
    if (tid == 0 && q + kNBuf < c.Q) issue_load<DT>(c, q + kNBuf);
    if (tid < SE) {
        float sum = 0.f;
#pragma unroll
        for (int g = 0; g < kRowGroups; ++g) sum += c.cs[g * SE + tid];
        const float m = sum / (float)p.f;
        c.mean_s[tid] = m;
        p.mean[(int64_t)t * p.d + s * SE + tid] = m;
    }
    __syncthreads();

    float2 negm[P / 2];
#pragma unroll
    for (int j = 0; j < P / 2; ++j) negm[j] = make_float2(-c.mean_s[v * P + 2 * j], -c.mean_s[v * P + 2 * j + 1]);

    float x[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) x[i] = 0.f;
    const float2 one = make_float2(1.f, 1.f), neg1 = make_float2(-1.f, -1.f);
#pragma unroll
    for (int r = 0; r < kRMax; ++r) {
        float a[P], b[P];
        E::widen(cur[r], a);
        float2 aa = make_float2(0.f, 0.f), dm = aa, db = aa, bb = aa;
#pragma unroll
        for (int j = 0; j < P / 2; ++j) {
            const float2 a2 = make_float2(a[2 * j], a[2 * j + 1]);
            const float2 e = ffma2(a2, one, negm[j]);           // a - m
            aa = ffma2(a2, a2, aa);
            dm = ffma2(e, e, dm);
        }
        if (!is_first) {
            E::widen(prev[r], b);
#pragma unroll
            for (int j = 0; j < P / 2; ++j) {
                const float2 a2 = make_float2(a[2 * j], a[2 * j + 1]);
                const float2 b2 = make_float2(b[2 * j], b[2 * j + 1]);
                const float2 e = ffma2(b2, neg1, a2);           // a - b
                db = ffma2(e, e, db);
                bb = ffma2(b2, b2, bb);
            }
        }
        x[4 * r + 0] = aa.x + aa.y;
        x[4 * r + 1] = dm.x + dm.y;
        x[4 * r + 2] = db.x + db.y;
        x[4 * r + 3] = bb.x + bb.y;
    }
    group16_reduce_scatter(x, v);
    {
        const int row = rg + kRowGroups * v;                    // lane v of the group holds row slot v
        if (v < kRMax && row < p.f) {
            float4* dst = reinterpret_cast<float4*>(p.part) + ((int64_t)t * p.nsl + s) * p.f + row;
            *dst = make_float4(x[0], x[1], x[2], x[3]);
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) c.flags[1] = (atomicAdd(p.counters + t, 1) == p.nsl - 1) ? 1 : 0;
    __syncthreads();
    if (c.flags[1]) {
        __threadfence();
        finalize_frame<DT>(c, t, is_first);
    }
    return true;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap tmap, const FusedParams p, int32_t* status_word) {
    constexpr int SE = Ctx<DT>::SE;
    extern __shared__ __align__(1024) unsigned char smem[];
    Ctx<DT> c;
    c.tmap = &tmap;
    c.p = &p;
    c.tiles = smem;
    unsigned char* after = smem + (size_t)kNBuf * p.tile_stride;
    c.cs = reinterpret_cast<float*>(after);
    c.mean_s = c.cs + kRowGroups * SE;
    c.fin = c.mean_s + SE;
    c.bars = reinterpret_cast<uint64_t*>(c.fin + 5 * kMaxTokensFused + 16);
    c.flags = reinterpret_cast<volatile int*>(c.bars + kNBuf);

    const int64_t U = (int64_t)p.nsl * p.F;
    c.u0 = U * blockIdx.x / gridDim.x;
    const int64_t u1 = U * (blockIdx.x + 1) / gridDim.x;
    if (c.u0 >= u1) return;
    c.halo = frame_is_first(p, (int)(c.u0 % p.F)) ? 0 : 1;
    c.Q = (int)(u1 - c.u0) + c.halo;

    const int tid = threadIdx.x, v = tid & 15, rg = tid >> 4;
    if (tid == 0) {
        for (int i = 0; i < kNBuf; ++i) mbar_init(c.bars + i, 1);
        c.flags[0] = 0;
        c.flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    int issued = 0;
    if (tid == 0) {
        for (; issued < kNBuf && issued < c.Q; ++issued) issue_load<DT>(c, issued);
    }

    uint4 A[kRMax], B[kRMax];
#pragma unroll
    for (int r = 0; r < kRMax; ++r) { A[r] = make_uint4(0u, 0u, 0u, 0u); B[r] = A[r]; }

    int q = 0;
    bool ok = true;
    if (c.halo) {                                       // frame before the first unit: registers only
        float unused[Ctx<DT>::P];
        tile_to_regs<DT>(c, 0, rg, v, B, unused);
        __syncthreads();
        ok = c.flags[0] == 0;
        if (ok && tid == 0 && kNBuf < c.Q) issue_load<DT>(c, kNBuf);
        q = 1;
    }
    int64_t u = c.u0;
    while (ok && u < u1) {
        ok = process_unit<DT>(c, q, (int)(u / p.F), (int)(u % p.F), A, B);
        ++q; ++u;
        if (!ok || u >= u1) break;
        ok = process_unit<DT>(c, q, (int)(u / p.F), (int)(u % p.F), B, A);
        ++q; ++u;
    }
    if (!ok) {
        // A wait on the CTA's own loads ran out.  Report it, then give the loads that are still in
        // flight one more bounded wait each, so that nothing lands in shared memory after exit.
        __syncthreads();
        if (tid == 0) {
            report(status_word, SHARPV_ERR_TIMEOUT);
            const int last = min(c.Q, q + kNBuf);
            for (int i = q; i < last; ++i) (void)mbar_wait(c.bars + (i % kNBuf), (uint32_t)((i / kNBuf) & 1));
        }
        __syncthreads();
    }
}

size_t smem_bytes(int f, int se) {
    const size_t tile_stride = align_up((size_t)f * kSliceBytes, 128);
    return kNBuf * tile_stride + (size_t)(kRowGroups * se + se + 5 * kMaxTokensFused + 16) * 4 + kNBuf * 8 + 16;
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
    const size_t smem = smem_bytes(a.f, Ctx<DT>::SE);
    if (cudaFuncSetAttribute(score_fused_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SHARPV_ERR_UNSUPPORTED;
    }
    if (cudaMemsetAsync(p.counters, 0, sizeof(int32_t) * (size_t)a.F, a.stream) != cudaSuccess) return SHARPV_ERR_CUDA;
    const int64_t units = (int64_t)p.nsl * a.F;
    const unsigned grid = (unsigned)(units < sms ? units : sms);
    score_fused_kernel<DT><<<grid, kThreads, smem, a.stream>>>(tmap, p, a.status_word);
    return launch_status();
}

}  // namespace

bool fused_score_supported(sharpv_dtype dtype, int f, int d) {
    const int64_t row_bytes = (int64_t)d * elem_bytes(dtype);
    return f >= 1 && f <= kMaxTokensFused && row_bytes % kSliceBytes == 0;
}

size_t fused_score_workspace_bytes(int F, int f, int d) {
    const size_t nsl_max = ((size_t)d * 4 + kSliceBytes - 1) / kSliceBytes;
    return align_up((size_t)F * d * 4, 256) + align_up((size_t)F * nsl_max * f * 16, 256) +
           align_up((size_t)F * 4, 256);
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
    p.part = (float*)w;       w += align_up((size_t)a.F * p.nsl * a.f * 16, 256);
    p.counters = (int32_t*)w;
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
