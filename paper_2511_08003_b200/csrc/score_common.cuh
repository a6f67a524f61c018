// Score arithmetic shared by the kernels of stage one (a): Dissim from row reductions, the
// exact re-evaluation for nearly parallel rows, and the budget rule (Eq. 1-6).
#pragma once

#include "common.cuh"

namespace sharpv {

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

// The same quantity from the inner product, 2 - 2 cos.  The cancellation leaves an absolute error of
// a few 1e-7, which is harmless for a token against its frame mean (far from parallel in practice);
// under kRefineBelowDot the caller re-evaluates from the rows.
__device__ __forceinline__ float dissim_sq_from_dot(float saa, float sbb, float sab) {
    const float na = sqrtf(saa), nb = sqrtf(sbb);
    if (na >= kNormEps && nb >= kNormEps) return fmaxf(2.f - 2.f * sab / (na * nb), 0.f);
    const float ca = fmaxf(na, kNormEps), cb = fmaxf(nb, kNormEps);
    return fmaxf(saa / (ca * ca) + sbb / (cb * cb) - 2.f * sab / (ca * cb), 0.f);
}

constexpr float kRefineBelowDot = 6.25e-2f;


// a * ca - b * cb with a single rounding of the difference: p = fl(a ca), e = a ca - p exactly (one
// fma), fl(p - b cb) by a second fma, then the exact error back in.  For nearly parallel rows the
// two products cancel to a few units in their last place; a plain fma(a, ca, -fl(b cb)) would
// leave the rounding of fl(b cb), which is as large as the difference itself.
__device__ __forceinline__ float scaled_difference(float a, float ca, float b, float cb) {
    const float p = a * ca;
    const float e = fmaf(a, ca, -p);
    return fmaf(-b, cb, p) + e;
}

// Exact re-evaluation of one token row: sums the squared differences of the normalised rows
// directly.  One warp per row; every lane returns the warp totals.  ia, ib, im are the
// reciprocal (clamped) norms of the row, of the previous-frame row and of the frame mean.
template <int DT>
__device__ __forceinline__ void refine_row(const char* pa, const char* pb, const float* pm, int nvec, int lane,
                                           bool refine_s, bool refine_t, float ia, float ib, float im,
                                           float& es_out, float& et_out) {
    using E = Elem<DT>;
    constexpr int P = E::kPerVec;
    float es = 0.f, et = 0.f;
    for (int v = lane; v < nvec; v += 32) {
        float a[P], b[P], m[P];
        E::widen(ld_cached(pa + (int64_t)v * 16), a);
        if (refine_s) {
#pragma unroll
            for (int j = 0; j < P; j += 4) {
                float4 q = __ldcg(reinterpret_cast<const float4*>(pm + (int64_t)v * P + j));
                m[j] = q.x; m[j + 1] = q.y; m[j + 2] = q.z; m[j + 3] = q.w;
            }
#pragma unroll
            for (int j = 0; j < P; ++j) {
                const float df = scaled_difference(a[j], ia, m[j], im);
                es = fmaf(df, df, es);
            }
        }
        if (refine_t) {
            E::widen(ld_cached(pb + (int64_t)v * 16), b);
#pragma unroll
            for (int j = 0; j < P; ++j) {
                const float df = scaled_difference(a[j], ia, b[j], ib);
                et = fmaf(df, df, et);
            }
        }
    }
    es_out = warp_sum(es);
    et_out = warp_sum(et);
}

// S, T and I of one token from the squared dissimilarities (Eq. 2-4)
__device__ __forceinline__ void scores_from_sq(float s2, float t2, bool is_first, int one_minus_cos, float w,
                                               float& S, float& T, float& I) {
    if (one_minus_cos) {            // 1 - cos = Dissim^2 / 2
        S = 0.5f * s2;
        T = is_first ? S : 0.5f * t2;
    } else {
        S = sqrtf(s2);
        T = is_first ? S : sqrtf(t2);
    }
    I = fmaf(w, S, T);
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


__device__ __forceinline__ float ratio_from_sumsq(float sum_t2, int f) {
    return sqrtf(sum_t2) / (2.f * sqrtf((float)f));
}

}  // namespace sharpv
