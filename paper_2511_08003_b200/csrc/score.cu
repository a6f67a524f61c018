// Stage one (a): spatial / temporal dissimilarity scores and the adaptive per-frame budget
// (Section 3.1.2 - 3.1.3, Eq. 1-6).
//
// Shapes that split into 128-byte column slices with frames of up to 256 tokens run in the single
// fused kernel of score_fused.cu.  Every other shape runs the three kernels below:
//   frame_mean_kernel   column sums of each frame -> frame mean (fp32), first-frame flags
//   row_scores_kernel   one warp per token: the row reductions behind S, T and I
//   frame_budget_kernel one CTA per frame: ||T_t||_2 -> ratio_t, k_t (fixed-order reduction)
#include "score_common.cuh"
#include "score_fused.cuh"

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
    // compensated (Kahan) column sums: the mean stays accurate to about one ulp however long the
    // frame is, which the spatial score of an almost uniform frame depends on; the kernel is
    // bandwidth-bound, so the extra adds are free
    float acc[P], comp[P];
#pragma unroll
    for (int j = 0; j < P; ++j) { acc[j] = 0.f; comp[j] = 0.f; }
    auto add_row = [&](const uint4& r) {
        float x[P];
        E::widen(r, x);
#pragma unroll
        for (int j = 0; j < P; ++j) {
            const float y = __fsub_rn(x[j], comp[j]);
            const float tsum = __fadd_rn(acc[j], y);
            comp[j] = __fsub_rn(__fsub_rn(tsum, acc[j]), y);
            acc[j] = tsum;
        }
    };
    int i = 0;
    for (; i + 4 <= f; i += 4) {
        uint4 r0 = ld_stream(base + (int64_t)(i + 0) * row_bytes_ld);
        uint4 r1 = ld_stream(base + (int64_t)(i + 1) * row_bytes_ld);
        uint4 r2 = ld_stream(base + (int64_t)(i + 2) * row_bytes_ld);
        uint4 r3 = ld_stream(base + (int64_t)(i + 3) * row_bytes_ld);
        add_row(r0); add_row(r1); add_row(r2); add_row(r3);
    }
    for (; i < f; ++i) add_row(ld_stream(base + (int64_t)i * row_bytes_ld));
    const float ff = (float)f;
    float* out = mean + (int64_t)t * d + (int64_t)v * P;
#pragma unroll
    for (int j = 0; j < P; j += 4) {
        float4 o = make_float4(acc[j] / ff, acc[j + 1] / ff, acc[j + 2] / ff, acc[j + 3] / ff);
        *reinterpret_cast<float4*>(out + j) = o;
    }
}

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
        float es, et;
        refine_row<DT>(pa, pb, pm, nvec, lane, refine_s, refine_t, ia, ib, im, es, et);
        if (refine_s) s2 = es;
        if (refine_t) t2 = et;
    }

    float S, T, I;
    scores_from_sq(s2, t2, is_first, one_minus_cos, w, S, T, I);
    if (lane == 0) {
        out_I[row] = I;
        if (out_S) out_S[row] = S;
        out_T[row] = T;
    }
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
        const float r = ratio_from_sumsq(tot, f);
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
    const size_t generic =
        ws_mean_bytes(total_frames, d) + ws_temporal_bytes(total_frames, f) + ws_first_bytes(total_frames);
    const size_t fused = fused_score_workspace_bytes(total_frames, f, d);
    return generic > fused ? generic : fused;
}

extern "C" sharpv_status sharpv_score_frames(
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t num_videos,
    const int32_t* video_frame_offsets, int32_t total_frames, int32_t f, int32_t d, float w,
    sharpv_dissim_kind dissim_kind, sharpv_round round_mode, int32_t min_keep, float* out_importance,
    float* out_spatial, float* out_temporal, float* out_ratio, int32_t* out_k, void* workspace,
    size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
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

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int omc = dissim_kind == SHARPV_ONE_MINUS_COS;
    if (fused_score_supported(dtype, f, d)) {
        FusedScoreArgs a;
        a.tokens = tokens; a.dtype = dtype; a.ld_tokens = ld_tokens; a.num_videos = num_videos;
        a.video_frame_offsets = video_frame_offsets; a.F = total_frames; a.f = f; a.d = d; a.w = w;
        a.one_minus_cos = omc; a.round_mode = (int)round_mode; a.min_keep = min_keep;
        a.out_I = out_importance; a.out_S = out_spatial; a.out_T = out_temporal; a.out_ratio = out_ratio;
        a.out_k = out_k; a.workspace = workspace; a.status_word = status_word; a.stream = stream;
        a.select = false; a.out_kept_index = nullptr; a.out_kept_offsets = nullptr; a.out_num_kept = nullptr;
        a.out_tokens = nullptr; a.capacity = 0;
        const sharpv_status st = fused_score_launch(a);
        if (st != SHARPV_ERR_UNSUPPORTED) return st;      // otherwise: set-up unavailable, use the generic kernels
    }

    ScoreWorkspace ws;
    char* p = (char*)workspace;
    ws.mean = (float*)p;       p += ws_mean_bytes(total_frames, d);
    ws.temporal = (float*)p;   p += ws_temporal_bytes(total_frames, f);
    ws.first = (int32_t*)p;
    if (dtype == SHARPV_F32)
        return launch_score<SHARPV_F32>(tokens, ld_tokens, num_videos, video_frame_offsets, total_frames, f, d,
                                        w, omc, (int)round_mode, min_keep, out_importance, out_spatial,
                                        out_temporal, out_ratio, out_k, ws, stream);
    return launch_score<SHARPV_BF16>(tokens, ld_tokens, num_videos, video_frame_offsets, total_frames, f, d, w,
                                     omc, (int)round_mode, min_keep, out_importance, out_spatial, out_temporal,
                                     out_ratio, out_k, ws, stream);
}


// ---------------------------------------------------------------------------------------
// Stage one in one call (Section 3.1): scores, budgets, per-frame top-k, gather.
// ---------------------------------------------------------------------------------------
namespace {
size_t prune_fused_bytes(int32_t F, int32_t f, int32_t d) {
    return fused_score_workspace_bytes(F, f, d) + fused_select_workspace_bytes(F, f);
}
}  // namespace

extern "C" size_t sharpv_prune_frames_workspace_bytes(int32_t total_frames, int32_t f, int32_t d) {
    if (total_frames <= 0 || f <= 0 || d <= 0) return 256;
    const size_t parts = sharpv_score_frames_workspace_bytes(total_frames, f, d) +
                         sharpv_select_tokens_workspace_bytes(total_frames, f);
    const size_t fused = prune_fused_bytes(total_frames, f, d);
    return parts > fused ? parts : fused;
}

extern "C" sharpv_status sharpv_prune_frames(
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t num_videos,
    const int32_t* video_frame_offsets, int32_t total_frames, int32_t f, int32_t d, float w,
    sharpv_dissim_kind dissim_kind, sharpv_round round_mode, int32_t min_keep, float* out_importance,
    float* out_spatial, float* out_temporal, float* out_ratio, int32_t* out_k, int32_t* out_kept_index,
    int32_t* out_kept_offsets, void* out_tokens, int64_t capacity, int32_t* out_num_kept, void* workspace,
    size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    if (!dtype_ok(dtype)) return SHARPV_ERR_UNSUPPORTED;
    if (num_videos < 1 || total_frames < 0 || f < 1 || d < 1 || min_keep < 0 || ld_tokens < d || capacity < 0)
        return SHARPV_ERR_INVALID_ARG;
    if ((int)round_mode < 0 || (int)round_mode > 2 || (int)dissim_kind < 0 || (int)dissim_kind > 1)
        return SHARPV_ERR_INVALID_ARG;
    if (!video_frame_offsets || !out_kept_offsets) return SHARPV_ERR_INVALID_ARG;
    if (capacity > 0 && !out_kept_index) return SHARPV_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (total_frames == 0) {
        if (cudaMemsetAsync(out_kept_offsets, 0, sizeof(int32_t), stream) != cudaSuccess) return SHARPV_ERR_CUDA;
        if (out_num_kept && cudaMemsetAsync(out_num_kept, 0, sizeof(int32_t), stream) != cudaSuccess)
            return SHARPV_ERR_CUDA;
        return SHARPV_OK;
    }
    if (!tokens || !out_importance || !out_ratio || !out_k || !workspace) return SHARPV_ERR_INVALID_ARG;
    if ((int64_t)total_frames * f >= (int64_t)1 << 31) return SHARPV_ERR_UNSUPPORTED;
    const int eb = elem_bytes(dtype);
    if (((int64_t)d * eb) % 16 || (ld_tokens * eb) % 16 || !aligned16(tokens) || !aligned16(workspace) ||
        (out_tokens && !aligned16(out_tokens)))
        return SHARPV_ERR_UNSUPPORTED;
    if (workspace_bytes < sharpv_prune_frames_workspace_bytes(total_frames, f, d)) return SHARPV_ERR_WORKSPACE;

    if (fused_score_supported(dtype, f, d)) {
        FusedScoreArgs a;
        a.tokens = tokens; a.dtype = dtype; a.ld_tokens = ld_tokens; a.num_videos = num_videos;
        a.video_frame_offsets = video_frame_offsets; a.F = total_frames; a.f = f; a.d = d; a.w = w;
        a.one_minus_cos = dissim_kind == SHARPV_ONE_MINUS_COS; a.round_mode = (int)round_mode; a.min_keep = min_keep;
        a.out_I = out_importance; a.out_S = out_spatial; a.out_T = out_temporal; a.out_ratio = out_ratio;
        a.out_k = out_k; a.workspace = workspace; a.status_word = status_word; a.stream = stream;
        a.select = true; a.out_kept_index = out_kept_index; a.out_kept_offsets = out_kept_offsets;
        a.out_num_kept = out_num_kept; a.out_tokens = out_tokens; a.capacity = capacity;
        const sharpv_status st = fused_score_launch(a);
        if (st != SHARPV_ERR_UNSUPPORTED) return st;      // otherwise: set-up unavailable, run the two entry points
    }
    // shapes outside the fused kernels: the two entry points one after the other
    const size_t score_bytes = sharpv_score_frames_workspace_bytes(total_frames, f, d);
    sharpv_status st = sharpv_score_frames(tokens, dtype, ld_tokens, num_videos, video_frame_offsets, total_frames, f, d,
                                           w, dissim_kind, round_mode, min_keep, out_importance, out_spatial,
                                           out_temporal, out_ratio, out_k, workspace, score_bytes, status_word,
                                           cuda_stream);
    if (st != SHARPV_OK) return st;
    return sharpv_select_tokens(out_importance, out_k, total_frames, f, tokens, dtype, ld_tokens, d, out_kept_index,
                                out_kept_offsets, out_tokens, capacity, out_num_kept, (char*)workspace + score_bytes,
                                workspace_bytes - score_bytes, status_word, cuda_stream);
}
