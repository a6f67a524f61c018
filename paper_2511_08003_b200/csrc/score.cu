// Stage one (a): spatial / temporal dissimilarity scores and the adaptive per-frame budget
// (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// Three kernels:
//   frame_mean_kernel   column sums of each frame -> frame mean (fp32), first-frame flags
//   row_scores_kernel   one warp per token: the row reductions behind S, T and I
//   frame_budget_kernel one CTA per frame: ||T_t||_2 -> ratio_t, k_t (fixed-order reduction)
#include "common.cuh"

namespace sharpv {
namespace {

struct ScoreWorkspace {
    float* mean;        // [F, d]
    float* temporal;    // [F * f] (used when the caller does not ask for T)
    int32_t* first;     // [F] 1 when the frame opens a video
};

__host__ __device__ inline size_t ws_mean_bytes(int F, int d) { return ((size_t)F * d * 4 + 255) / 256 * 256; }
__host__ __device__ inline size_t ws_temporal_bytes(int F, int f) { return ((size_t)F * f * 4 + 255) / 256 * 256; }
__host__ __device__ inline size_t ws_first_bytes(int F) { return ((size_t)F * 4 + 255) / 256 * 256; }

// ---------------------------------------------------------------------------------------
// frame mean: thread owns one 16-byte column group, walks the f rows of the frame
// ---------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(128)
frame_mean_kernel(const char* __restrict__ tokens, int64_t row_bytes_ld, int f, int d, int nvec,
                  int num_videos, const int32_t* __restrict__ video_frame_offsets,
                  float* __restrict__ mean, int32_t* __restrict__ first) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    const int t = blockIdx.x;
    const int v = blockIdx.y * blockDim.x + threadIdx.x;
    if (blockIdx.y == 0 && threadIdx.x == 0) {
        int b = upper_segment(video_frame_offsets, num_videos, t);
        first[t] = (__ldg(video_frame_offsets + b) == t) ? 1 : 0;
    }
    if (v >= nvec) return;
    const char* base = tokens + (int64_t)t * f * row_bytes_ld + (int64_t)v * 16;
    float acc[P];
#pragma unroll
    for (int j = 0; j < P; ++j) acc[j] = 0.f;
    int i = 0;
    for (; i + 4 <= f; i += 4) {
        uint4 r0 = ld_stream(base + (int64_t)(i + 0) * row_bytes_ld);
        uint4 r1 = ld_stream(base + (int64_t)(i + 1) * row_bytes_ld);
        uint4 r2 = ld_stream(base + (int64_t)(i + 2) * row_bytes_ld);
        uint4 r3 = ld_stream(base + (int64_t)(i + 3) * row_bytes_ld);
        float x[P];
        E::widen(r0, x);
#pragma unroll
        for (int j = 0; j < P; ++j) acc[j] += x[j];
        E::widen(r1, x);
#pragma unroll
        for (int j = 0; j < P; ++j) acc[j] += x[j];
        E::widen(r2, x);
#pragma unroll
        for (int j = 0; j < P; ++j) acc[j] += x[j];
        E::widen(r3, x);
#pragma unroll
        for (int j = 0; j < P; ++j) acc[j] += x[j];
    }
    for (; i < f; ++i) {
        uint4 r0 = ld_stream(base + (int64_t)i * row_bytes_ld);
        float x[P];
        E::widen(r0, x);
#pragma unroll
        for (int j = 0; j < P; ++j) acc[j] += x[j];
    }
    const float ff = (float)f;
    float* out = mean + (int64_t)t * d + (int64_t)v * P;
#pragma unroll
    for (int j = 0; j < P; j += 4) {
        float4 o = make_float4(acc[j] / ff, acc[j + 1] / ff, acc[j + 2] / ff, acc[j + 3] / ff);
        *reinterpret_cast<float4*>(out + j) = o;
    }
}

// ---------------------------------------------------------------------------------------
// Dissim from row reductions.
//   ||a^ - b^||^2 = (||a-b||^2 - (||a|| - ||b||)^2) / (||a|| ||b||)
// is algebraically 2 - 2 cos but has no cancellation for nearly parallel rows and is exactly
// zero for identical rows.  Rows that are nearly parallel without being close (b ~ alpha a,
// or a token next to a mean of identical tokens) are re-evaluated by the caller from the
// normalised rows themselves.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float dissim_sq_from_sums(float saa, float sbb, float sdd) {
    const float na = sqrtf(saa), nb = sqrtf(sbb);
    if (na >= kNormEps && nb >= kNormEps) {
        const float dn = na - nb;
        return fmaxf(sdd - dn * dn, 0.f) / (na * nb);
    }
    // at least one (near-)zero vector: v^ = v / max(||v||, eps)
    const float ca = fmaxf(na, kNormEps), cb = fmaxf(nb, kNormEps);
    const float sab = 0.5f * (saa + sbb - sdd);
    return fmaxf(saa / (ca * ca) + sbb / (cb * cb) - 2.f * sab / (ca * cb), 0.f);
}

constexpr float kRefineBelow = 1e-2f;   // squared Dissim under which the exact form is used

template <int DT>
__global__ void __launch_bounds__(256)
row_scores_kernel(const char* __restrict__ tokens, int64_t row_bytes_ld, int f, int d, int nvec,
                  int64_t n_rows, const float* __restrict__ mean, const int32_t* __restrict__ first,
                  float w, int one_minus_cos,
                  float* __restrict__ out_I, float* __restrict__ out_S, float* __restrict__ out_T) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const int t = (int)(row / f);
    const bool is_first = __ldg(first + t) != 0;
    const char* pa = tokens + row * row_bytes_ld;
    const char* pb = pa - (int64_t)f * row_bytes_ld;
    const float* pm = mean + (int64_t)t * d;

    float saa = 0.f, sbb = 0.f, sdd = 0.f, smm = 0.f, sdm = 0.f;
    for (int v = lane; v < nvec; v += 32) {
        float a[P], b[P], m[P];
        E::widen(ld_stream(pa + (int64_t)v * 16), a);
#pragma unroll
        for (int j = 0; j < P; j += 4) {
            float4 q = __ldg(reinterpret_cast<const float4*>(pm + (int64_t)v * P + j));
            m[j] = q.x; m[j + 1] = q.y; m[j + 2] = q.z; m[j + 3] = q.w;
        }
        if (!is_first) {
            E::widen(ld_stream(pb + (int64_t)v * 16), b);
#pragma unroll
            for (int j = 0; j < P; ++j) {
                const float df = a[j] - b[j];
                sbb = fmaf(b[j], b[j], sbb);
                sdd = fmaf(df, df, sdd);
            }
        }
#pragma unroll
        for (int j = 0; j < P; ++j) {
            const float dm = a[j] - m[j];
            saa = fmaf(a[j], a[j], saa);
            smm = fmaf(m[j], m[j], smm);
            sdm = fmaf(dm, dm, sdm);
        }
    }
    saa = warp_sum(saa); sbb = warp_sum(sbb); sdd = warp_sum(sdd);
    smm = warp_sum(smm); sdm = warp_sum(sdm);

    // every lane holds the same sums from here on: the branches below are warp-uniform
    float s2 = dissim_sq_from_sums(saa, smm, sdm);
    float t2 = is_first ? 0.f : dissim_sq_from_sums(saa, sbb, sdd);

    const float na = fmaxf(sqrtf(saa), kNormEps);
    const bool refine_s = s2 < kRefineBelow && sdm != 0.f;
    const bool refine_t = !is_first && t2 < kRefineBelow && sdd != 0.f;
    if (refine_s || refine_t) {
        // nearly parallel rows: sum the squared differences of the normalised rows directly
        const float ia = 1.f / na;
        const float im = 1.f / fmaxf(sqrtf(smm), kNormEps);
        const float ib = 1.f / fmaxf(sqrtf(sbb), kNormEps);
        float es = 0.f, et = 0.f;
        for (int v = lane; v < nvec; v += 32) {
            float a[P], b[P], m[P];
            E::widen(ld_cached(pa + (int64_t)v * 16), a);
            if (refine_s) {
#pragma unroll
                for (int j = 0; j < P; j += 4) {
                    float4 q = __ldg(reinterpret_cast<const float4*>(pm + (int64_t)v * P + j));
                    m[j] = q.x; m[j + 1] = q.y; m[j + 2] = q.z; m[j + 3] = q.w;
                }
#pragma unroll
                for (int j = 0; j < P; ++j) {
                    const float df = fmaf(a[j], ia, -m[j] * im);
                    es = fmaf(df, df, es);
                }
            }
            if (refine_t) {
                E::widen(ld_cached(pb + (int64_t)v * 16), b);
#pragma unroll
                for (int j = 0; j < P; ++j) {
                    const float df = fmaf(a[j], ia, -b[j] * ib);
                    et = fmaf(df, df, et);
                }
            }
        }
        es = warp_sum(es); et = warp_sum(et);
        if (refine_s) s2 = es;
        if (refine_t) t2 = et;
    }

    float S, T;
    if (one_minus_cos) {            // 1 - cos = Dissim^2 / 2
        S = 0.5f * s2;
        T = is_first ? S : 0.5f * t2;
    } else {
        S = sqrtf(s2);
        T = is_first ? S : sqrtf(t2);
    }
    if (lane == 0) {
        out_I[row] = fmaf(w, S, T);
        if (out_S) out_S[row] = S;
        out_T[row] = T;
    }
}

// ---------------------------------------------------------------------------------------
// per-frame budget: ratio_t = ||T_t||_2 / (2 sqrt(f)), k_t = clamp(round(ratio_t f))
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int budget_from_ratio(float r, int f, int round_mode, int min_keep) {
    const float x = r * (float)f;
    float y;
    if (round_mode == SHARPV_ROUND_FLOOR) y = floorf(x);
    else if (round_mode == SHARPV_ROUND_NEAREST) y = floorf(x + 0.5f);
    else y = ceilf(x);
    int k = (int)y;
    k = max(k, min_keep);
    k = min(k, f);
    return max(k, 0);
}

__global__ void __launch_bounds__(256)
frame_budget_kernel(const float* __restrict__ temporal, int f, int round_mode, int min_keep,
                    float* __restrict__ out_ratio, int32_t* __restrict__ out_k) {
    __shared__ float part[8];
    const int t = blockIdx.x;
    const float* T = temporal + (int64_t)t * f;
    float s = 0.f;
    for (int i = threadIdx.x; i < f; i += 256) {
        const float x = T[i];
        s = fmaf(x, x, s);
    }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += part[i];
        const float r = sqrtf(tot) / (2.f * sqrtf((float)f));
        out_ratio[t] = r;
        out_k[t] = budget_from_ratio(r, f, round_mode, min_keep);
    }
}

template <int DT>
sharpv_status launch_score(const void* tokens, int64_t ld_tokens, int num_videos,
                           const int32_t* video_frame_offsets, int F, int f, int d, float w,
                           int one_minus_cos, int round_mode, int min_keep, float* out_I, float* out_S,
                           float* out_T, float* out_ratio, int32_t* out_k, const ScoreWorkspace& ws,
                           cudaStream_t stream) {
    constexpr int EB = Elem<DT>::kBytes;
    const int nvec = d * EB / 16;
    const int64_t row_bytes_ld = ld_tokens * EB;
    dim3 g1(F, (nvec + 127) / 128);
    frame_mean_kernel<DT><<<g1, 128, 0, stream>>>((const char*)tokens, row_bytes_ld, f, d, nvec, num_videos,
                                                  video_frame_offsets, ws.mean, ws.first);
    const int64_t n_rows = (int64_t)F * f;
    float* T = out_T ? out_T : ws.temporal;
    row_scores_kernel<DT><<<(unsigned)((n_rows + 7) / 8), 256, 0, stream>>>(
        (const char*)tokens, row_bytes_ld, f, d, nvec, n_rows, ws.mean, ws.first, w, one_minus_cos,
        out_I, out_S, T);
    frame_budget_kernel<<<F, 256, 0, stream>>>(T, f, round_mode, min_keep, out_ratio, out_k);
    return launch_status();
}

}  // namespace
}  // namespace sharpv

using namespace sharpv;

extern "C" size_t sharpv_score_frames_workspace_bytes(int32_t total_frames, int32_t f, int32_t d) {
    if (total_frames <= 0 || f <= 0 || d <= 0) return 256;
    return ws_mean_bytes(total_frames, d) + ws_temporal_bytes(total_frames, f) + ws_first_bytes(total_frames);
}

extern "C" sharpv_status sharpv_score_frames(
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t num_videos,
    const int32_t* video_frame_offsets, int32_t total_frames, int32_t f, int32_t d, float w,
    sharpv_dissim_kind dissim_kind, sharpv_round round_mode, int32_t min_keep, float* out_importance,
    float* out_spatial, float* out_temporal, float* out_ratio, int32_t* out_k, void* workspace,
    size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    (void)status_word;
    if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (num_videos < 1 || total_frames < 0 || f < 1 || d < 1 || min_keep < 0 || ld_tokens < d)
        return SHARPV_ERR_INVALID_ARG;
    if ((int)round_mode < 0 || (int)round_mode > 2 || (int)dissim_kind < 0 || (int)dissim_kind > 1)
        return SHARPV_ERR_INVALID_ARG;
    if (!video_frame_offsets) return SHARPV_ERR_INVALID_ARG;
    if (total_frames == 0) return SHARPV_OK;
    if (!tokens || !out_importance || !out_ratio || !out_k || !workspace) return SHARPV_ERR_INVALID_ARG;
    if ((int64_t)total_frames * f >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    const int eb = elem_bytes(dtype);
    if (((int64_t)d * eb) % 16 || (ld_tokens * eb) % 16 || !aligned16(tokens) || !aligned16(workspace))
        return SHARPV_ERR_UNSUPPORTED;
    if (workspace_bytes < sharpv_score_frames_workspace_bytes(total_frames, f, d)) return SHARPV_ERR_WORKSPACE;

    ScoreWorkspace ws;
    char* p = (char*)workspace;
    ws.mean = (float*)p;       p += ws_mean_bytes(total_frames, d);
    ws.temporal = (float*)p;   p += ws_temporal_bytes(total_frames, f);
    ws.first = (int32_t*)p;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int omc = dissim_kind == SHARPV_ONE_MINUS_COS;
    if (dtype == SHARPV_F32)
        return launch_score<SHARPV_F32>(tokens, ld_tokens, num_videos, video_frame_offsets, total_frames, f, d,
                                        w, omc, (int)round_mode, min_keep, out_importance, out_spatial,
                                        out_temporal, out_ratio, out_k, ws, stream);
    return launch_score<SHARPV_BF16>(tokens, ld_tokens, num_videos, video_frame_offsets, total_frames, f, d, w,
                                     omc, (int)round_mode, min_keep, out_importance, out_spatial, out_temporal,
                                     out_ratio, out_k, ws, stream);
}
