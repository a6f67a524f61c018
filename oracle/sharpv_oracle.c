/*
 * SharpV oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of what the SharpV pruning path
 * computes (arxiv 2511.08003, Sections 3.1 and 3.2).  It exists so that the CUDA
 * library can be checked against something written directly from the paper.  It
 * shares no code with the CUDA library and must never be called from it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every floating-point quantity is accumulated in double from inputs widened
 * exactly (fp32 or bf16 -> double).  Loops follow the paper's equations one to
 * one: no blocking, no fusion, no reordering.  `nthreads` only splits the
 * outermost independent loop (frames, tokens, planes) with OpenMP.
 *
 * Integer decisions that depend on a floating-point value (the per-frame budget
 * k_t, the order of scores, the test cos >= M) are taken on the value rounded to
 * fp32, the precision in which the library takes them.
 *
 * Readings of the paper where it is silent (each is a convention; the tests pin
 * the arithmetic around them, not the choice itself):
 *   - first frame of a video: T_1 := S_1 (Section 3.1.3 treats the first frame as if a frame made
 *     of its own mean stood in front of it), so Eq. 6 is Eq. 5 applied to that T_1;
 *   - the threshold of Eq. 5/6 is a retention ratio: k_t = round(threshold_t * f)
 *     followed by a per-frame top-k_t on I (Section 3.1.3, last paragraph);
 *   - ties in the top-k go to the lower token index; kept indices are reported
 *     in ascending order;
 *   - a zero vector normalises to zero: v^ = v / max(||v||, 1e-12);
 *   - Eq. 7 is applied per visual token at one layer; a token is kept iff
 *     cos >= M; tokens that are not visual are always kept.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_EPS 1e-12

static double load_elem(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

static void load_row(const void *base, int dtype, int64_t row, int64_t ld, int d, double *out)
{
    for (int j = 0; j < d; ++j)
        out[j] = load_elem(base, dtype, row * ld + j);
}

static double norm2(const double *v, int d)
{
    double s = 0.0;
    for (int j = 0; j < d; ++j)
        s += v[j] * v[j];
    return sqrt(s);
}

/* Eq. 1, left-hand side taken literally: the Euclidean distance between the two
 * L2-normalised vectors. */
double sharpv_oracle_dissim(const double *v1, const double *v2, int d)
{
    double n1 = fmax(norm2(v1, d), ORACLE_EPS);
    double n2 = fmax(norm2(v2, d), ORACLE_EPS);
    double s = 0.0;
    for (int j = 0; j < d; ++j) {
        double diff = v1[j] / n1 - v2[j] / n2;
        s += diff * diff;
    }
    return sqrt(s);
}

/* Cosine similarity of Eq. 7: inner product of the two normalised vectors. */
double sharpv_oracle_cosine(const double *v1, const double *v2, int d)
{
    double n1 = fmax(norm2(v1, d), ORACLE_EPS);
    double n2 = fmax(norm2(v2, d), ORACLE_EPS);
    double s = 0.0;
    for (int j = 0; j < d; ++j)
        s += (v1[j] / n1) * (v2[j] / n2);
    return s;
}

/* Manual variant's dissimilarity (Section 3.1.1, last sentence): 1 - cos. */
double sharpv_oracle_one_minus_cos(const double *v1, const double *v2, int d)
{
    return 1.0 - sharpv_oracle_cosine(v1, v2, d);
}

static int budget_from_ratio(double r, int f, int round_mode, int min_keep)
{
    float x = (float)r * (float)f;
    float y;
    if (round_mode == 0)
        y = floorf(x);
    else if (round_mode == 1)
        y = floorf(x + 0.5f);
    else
        y = ceilf(x);
    int k = (int)y;
    if (k < min_keep) k = min_keep;
    if (k > f) k = f;
    if (k < 0) k = 0;
    return k;
}

/*
 * Stage one, scores and budgets (Section 3.1.2 and 3.1.3, Eq. 2-6).
 * tokens: [total_frames*f, d] with row stride ld (elements).
 * dissim_kind: 0 = Dissim of Eq. 1, 1 = (1 - cos) (manual variant).
 * Outputs (double): spatial, temporal, importance [total_frames*f]; ratio [total_frames];
 * k [total_frames] (int32).  Returns 0, or -1 on a bad argument / failed allocation.
 */
int sharpv_oracle_score_frames(const void *tokens, int dtype, int64_t ld,
                               int num_videos, const int32_t *video_frame_offsets,
                               int f, int d, double w, int round_mode, int min_keep, int dissim_kind,
                               double *spatial, double *temporal, double *importance,
                               double *ratio, int32_t *k, int nthreads)
{
    if (!tokens || !video_frame_offsets || num_videos < 1 || f < 1 || d < 1)
        return -1;
    if (nthreads < 1) nthreads = 1;
    int total_frames = video_frame_offsets[num_videos];
    int *first = (int *)calloc((size_t)(total_frames > 0 ? total_frames : 1), sizeof(int));
    if (!first) return -1;
    for (int b = 0; b < num_videos; ++b)
        if (video_frame_offsets[b] < video_frame_offsets[b + 1])
            first[video_frame_offsets[b]] = 1;
    int fail = 0;

#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
    for (int t = 0; t < total_frames; ++t) {
        double *mean = (double *)malloc(sizeof(double) * (size_t)d);
        double *cur = (double *)malloc(sizeof(double) * (size_t)d);
        double *prev = (double *)malloc(sizeof(double) * (size_t)d);
        if (!mean || !cur || !prev) {
            fail = 1;
            free(mean); free(cur); free(prev);
            continue;
        }
        /* frame mean, Section 3.1.2 */
        for (int j = 0; j < d; ++j) mean[j] = 0.0;
        for (int i = 0; i < f; ++i) {
            load_row(tokens, dtype, (int64_t)t * f + i, ld, d, cur);
            for (int j = 0; j < d; ++j) mean[j] += cur[j];
        }
        for (int j = 0; j < d; ++j) mean[j] /= (double)f;

        double sumsq = 0.0;
        for (int i = 0; i < f; ++i) {
            int64_t row = (int64_t)t * f + i;
            load_row(tokens, dtype, row, ld, d, cur);
            double S = dissim_kind == 0 ? sharpv_oracle_dissim(cur, mean, d)
                                        : sharpv_oracle_one_minus_cos(cur, mean, d);   /* Eq. 2 */
            double T;
            if (first[t]) {
                T = S;                                                                /* Sec. 3.1.3 */
            } else {
                load_row(tokens, dtype, row - f, ld, d, prev);
                T = dissim_kind == 0 ? sharpv_oracle_dissim(cur, prev, d)
                                     : sharpv_oracle_one_minus_cos(cur, prev, d);      /* Eq. 3 */
            }
            if (spatial) spatial[row] = S;
            if (temporal) temporal[row] = T;
            if (importance) importance[row] = T + w * S;                              /* Eq. 4 */
            sumsq += T * T;
        }
        double r = sqrt(sumsq) / (2.0 * sqrt((double)f));                             /* Eq. 5, 6 */
        if (ratio) ratio[t] = r;
        if (k) k[t] = budget_from_ratio(r, f, round_mode, min_keep);
        free(mean); free(cur); free(prev);
    }
    free(first);
    return fail ? -1 : 0;
}

/*
 * Stage one, selection: in each frame keep the k_t tokens that come first under
 * "importance descending, then index ascending" (importance compared in fp32).
 * A token's rank is the number of tokens of its frame that precede it in that
 * order; it is kept iff rank < k_t.  kept_index: global token indices, ascending;
 * kept_offsets[F+1]: exclusive scan of k.  Returns the number kept.
 */
int64_t sharpv_oracle_select_tokens(const float *importance, const int32_t *k,
                                    int total_frames, int f,
                                    int32_t *kept_index, int32_t *kept_offsets)
{
    int64_t n = 0;
    for (int t = 0; t < total_frames; ++t) {
        kept_offsets[t] = (int32_t)n;
        const float *s = importance + (int64_t)t * f;
        int kt = k[t] < 0 ? 0 : (k[t] > f ? f : k[t]);
        for (int i = 0; i < f; ++i) {
            int rank = 0;
            for (int j = 0; j < f; ++j)
                if (s[j] > s[i] || (s[j] == s[i] && j < i))
                    ++rank;
            if (rank < kt)
                kept_index[n++] = (int32_t)((int64_t)t * f + i);
        }
    }
    kept_offsets[total_frames] = (int32_t)n;
    return n;
}

/* Manual variant: keep every token whose importance (fp32) exceeds the fixed cut K. */
int64_t sharpv_oracle_select_threshold(const float *importance, float K,
                                       int total_frames, int f,
                                       int32_t *kept_index, int32_t *kept_offsets)
{
    int64_t n = 0;
    for (int t = 0; t < total_frames; ++t) {
        kept_offsets[t] = (int32_t)n;
        for (int i = 0; i < f; ++i)
            if (importance[(int64_t)t * f + i] > K)
                kept_index[n++] = (int32_t)((int64_t)t * f + i);
    }
    kept_offsets[total_frames] = (int32_t)n;
    return n;
}

/* dst[j, :] = src[index[j], :], rows of row_bytes bytes, strides in bytes. */
void sharpv_oracle_gather_rows(const void *src, int64_t src_stride_bytes, int64_t row_bytes,
                               const int32_t *index, int64_t n, void *dst, int64_t dst_stride_bytes)
{
    for (int64_t j = 0; j < n; ++j)
        memcpy((char *)dst + j * dst_stride_bytes,
               (const char *)src + (int64_t)index[j] * src_stride_bytes, (size_t)row_bytes);
}

/*
 * Stage two, calibration (Section 3.2.3, Eq. 7), per visual token.
 * Sequence b owns hidden rows [seq_offsets[b], seq_offsets[b+1]); its visual
 * tokens are the vis_count[b] rows from seq_offsets[b] + vis_begin[b]; they map
 * in order to rows vis_offsets[b].. of the visual matrix.
 * cos_out [total_visual] (double); kept_pos: kept packed positions, ascending;
 * kept_seq_offsets [B+1].  Returns the number kept or -1.
 */
int64_t sharpv_oracle_kv_calibrate_prune(const void *hidden, int64_t ld_hidden,
                                         const void *visual, int64_t ld_visual, int dtype, int d,
                                         int num_seqs, const int32_t *seq_offsets,
                                         const int32_t *vis_begin, const int32_t *vis_count,
                                         const int32_t *vis_offsets, double M,
                                         double *cos_out, int32_t *kept_pos,
                                         int32_t *kept_seq_offsets, int nthreads)
{
    if (!hidden || !visual || !seq_offsets || num_seqs < 1 || d < 1) return -1;
    if (nthreads < 1) nthreads = 1;
    int64_t T = seq_offsets[num_seqs];
    unsigned char *keep = (unsigned char *)malloc((size_t)(T > 0 ? T : 1));
    if (!keep) return -1;
    memset(keep, 1, (size_t)(T > 0 ? T : 1));       /* non-visual tokens are never pruned */
    int fail = 0;
    for (int b = 0; b < num_seqs; ++b) {
        int64_t base = (int64_t)seq_offsets[b] + vis_begin[b];
#pragma omp parallel for num_threads(nthreads) schedule(static)
        for (int i = 0; i < vis_count[b]; ++i) {
            double *h = (double *)malloc(sizeof(double) * (size_t)d);
            double *v = (double *)malloc(sizeof(double) * (size_t)d);
            if (!h || !v) { fail = 1; free(h); free(v); continue; }
            load_row(hidden, dtype, base + i, ld_hidden, d, h);
            load_row(visual, dtype, (int64_t)vis_offsets[b] + i, ld_visual, d, v);
            double c = sharpv_oracle_cosine(h, v, d);
            if (cos_out) cos_out[(int64_t)vis_offsets[b] + i] = c;
            keep[base + i] = ((float)c < (float)M) ? 0 : 1;      /* Eq. 7: discard iff cos < M */
            free(h); free(v);
        }
    }
    int64_t n = 0;
    for (int b = 0; b < num_seqs; ++b) {
        kept_seq_offsets[b] = (int32_t)n;
        for (int64_t p = seq_offsets[b]; p < seq_offsets[b + 1]; ++p)
            if (keep[p]) kept_pos[n++] = (int32_t)p;
    }
    kept_seq_offsets[num_seqs] = (int32_t)n;
    free(keep);
    return fail ? -1 : n;
}

/*
 * Stage two read as Eq. 7 is printed (Section 3.2.3): Discard = cos(V_l, V) < M is one decision per
 * layer l, taken on the similarity between the layer's visual hidden states V_l and the original
 * visual features V; the similarity of two token matrices is the average of the token-wise cosines
 * (the per-layer average similarity of Section 3.2.1, Fig. 3), taken per sequence.  A layer that
 * fails the test loses the K/V of its visual tokens, and so does every deeper layer ("hierarchical"
 * pruning, Section 1; Section 4.3.2 counts the layers below the threshold); text tokens are never
 * dropped.
 *   hidden: n_layers hidden states, layer i at hidden + i * stride_layer elements, each [T, d];
 *   mean_cos [n_layers * B]: average cosine of sequence b at layer i (0 for a sequence without
 *     visual tokens);
 *   first_discard [B]: the first layer index i with mean_cos < M (decided in fp32), n_layers if none;
 *   per layer i: kept_pos + i * T (ascending packed positions) and kept_seq_offsets + i * (B + 1).
 * Returns 0 or -1.
 */
int sharpv_oracle_kv_discard_layers(const void *hidden, int64_t stride_layer, int64_t ld_hidden,
                                    const void *visual, int64_t ld_visual, int dtype, int d,
                                    int n_layers, int num_seqs, const int32_t *seq_offsets,
                                    const int32_t *vis_begin, const int32_t *vis_count,
                                    const int32_t *vis_offsets, double M,
                                    double *mean_cos, int32_t *first_discard,
                                    int32_t *kept_pos, int32_t *kept_seq_offsets, int nthreads)
{
    if (!hidden || !visual || !seq_offsets || num_seqs < 1 || d < 1 || n_layers < 0) return -1;
    if (nthreads < 1) nthreads = 1;
    int64_t T = seq_offsets[num_seqs];
    int fail = 0;
    for (int b = 0; b < num_seqs; ++b) first_discard[b] = n_layers;
    for (int i = 0; i < n_layers; ++i) {
        for (int b = 0; b < num_seqs; ++b) {
            int64_t base = (int64_t)seq_offsets[b] + vis_begin[b];
            double sum = 0.0;
#pragma omp parallel for num_threads(nthreads) schedule(static) reduction(+ : sum)
            for (int r = 0; r < vis_count[b]; ++r) {
                double *h = (double *)malloc(sizeof(double) * (size_t)d);
                double *v = (double *)malloc(sizeof(double) * (size_t)d);
                if (!h || !v) { fail = 1; free(h); free(v); continue; }
                /* layer i starts stride_layer elements further on */
                for (int j = 0; j < d; ++j)
                    h[j] = load_elem(hidden, dtype, (int64_t)i * stride_layer + (base + r) * ld_hidden + j);
                load_row(visual, dtype, (int64_t)vis_offsets[b] + r, ld_visual, d, v);
                sum += sharpv_oracle_cosine(h, v, d);
                free(h); free(v);
            }
            double mean = vis_count[b] > 0 ? sum / (double)vis_count[b] : 0.0;
            mean_cos[(int64_t)i * num_seqs + b] = mean;
            if (vis_count[b] > 0 && first_discard[b] == n_layers && (float)mean < (float)M)
                first_discard[b] = i;                       /* Eq. 7, and every deeper layer with it */
        }
        int32_t *kp = kept_pos + (int64_t)i * T;
        int32_t *kso = kept_seq_offsets + (int64_t)i * (num_seqs + 1);
        int64_t n = 0;
        for (int b = 0; b < num_seqs; ++b) {
            kso[b] = (int32_t)n;
            int dropped = i >= first_discard[b];
            int64_t v0 = (int64_t)seq_offsets[b] + vis_begin[b], v1 = v0 + vis_count[b];
            for (int64_t p = seq_offsets[b]; p < seq_offsets[b + 1]; ++p)
                if (!(dropped && p >= v0 && p < v1)) kp[n++] = (int32_t)p;
        }
        kso[num_seqs] = (int32_t)n;
    }
    return fail ? -1 : 0;
}

/*
 * Stage two, K/V compaction: for every layer in [layer_begin, layer_end), K and V,
 * and KV head, dst[j, :] = src[kept_pos[j], :] for j < n_kept.  Strides in bytes;
 * the head_dim axis is contiguous (row_bytes bytes).
 */
void sharpv_oracle_kv_compact(const void *src, void *dst, int num_kv_heads, int64_t row_bytes,
                              int64_t src_stride_layer, int64_t src_stride_kv,
                              int64_t src_stride_head, int64_t src_stride_token,
                              int64_t dst_stride_layer, int64_t dst_stride_kv,
                              int64_t dst_stride_head, int64_t dst_stride_token,
                              int layer_begin, int layer_end,
                              const int32_t *kept_pos, int64_t n_kept, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    int planes = (layer_end - layer_begin) * 2 * num_kv_heads;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int p = 0; p < planes; ++p) {
        int l = layer_begin + p / (2 * num_kv_heads);
        int kv = (p / num_kv_heads) % 2;
        int h = p % num_kv_heads;
        const char *s = (const char *)src + l * src_stride_layer + kv * src_stride_kv + h * src_stride_head;
        char *o = (char *)dst + l * dst_stride_layer + kv * dst_stride_kv + h * dst_stride_head;
        for (int64_t j = 0; j < n_kept; ++j)
            memcpy(o + j * dst_stride_token, s + (int64_t)kept_pos[j] * src_stride_token, (size_t)row_bytes);
    }
}

/*
 * In-place variant of the K/V compaction: within every plane, row j becomes the old row kept_pos[j]
 * for j < n_kept, everything behind stays as it was.  Written as "copy the plane, then gather from
 * the copy", which is the definition and cannot alias.
 */
int sharpv_oracle_kv_compact_inplace(void *kv, int num_kv_heads, int64_t row_bytes,
                                     int64_t stride_layer, int64_t stride_kv, int64_t stride_head,
                                     int64_t stride_token, int64_t tokens, int layer_begin, int layer_end,
                                     const int32_t *kept_pos, int64_t n_kept)
{
    int planes = (layer_end - layer_begin) * 2 * num_kv_heads;
    char *copy = (char *)malloc((size_t)(tokens > 0 ? tokens : 1) * (size_t)row_bytes);
    if (!copy) return -1;
    for (int p = 0; p < planes; ++p) {
        int l = layer_begin + p / (2 * num_kv_heads);
        int kv_i = (p / num_kv_heads) % 2;
        int h = p % num_kv_heads;
        char *base = (char *)kv + l * stride_layer + kv_i * stride_kv + h * stride_head;
        for (int64_t t = 0; t < tokens; ++t)
            memcpy(copy + t * row_bytes, base + t * stride_token, (size_t)row_bytes);
        for (int64_t j = 0; j < n_kept; ++j)
            memcpy(base + j * stride_token, copy + (int64_t)kept_pos[j] * row_bytes, (size_t)row_bytes);
    }
    free(copy);
    return 0;
}

/*
 * K/V compaction with positional re-encoding (Section 4.1.4: the positional embedding is encoded
 * again when Memory SharpV prunes inside the LLM).  Reading, the paper giving no detail: the cached
 * keys carry a rotary embedding of their old position (half-split pairing: dimension i pairs with
 * i + rotary_dim/2, angle position * base^(-2i/rotary_dim)); a kept token moves from position
 * p_old = kept_pos[j] - seq_offsets[b] to p_new = j - kept_seq_offsets[b] inside its sequence b, so
 * its key is rotated by (p_new - p_old): x1' = x1 cos - x2 sin, x2' = x2 cos + x1 sin.  Values and
 * the dimensions beyond rotary_dim are copied unchanged.  Output in double (the caller compares
 * with the storage rounding in mind).  out: [L', 2, H, n_kept, D_h] dense, L' = layer_end - layer_begin.
 */
int sharpv_oracle_kv_compact_rope(const void *src, int dtype, int num_kv_heads, int head_dim,
                                  int64_t stride_layer, int64_t stride_kv, int64_t stride_head,
                                  int64_t stride_token, int layer_begin, int layer_end,
                                  const int32_t *kept_pos, const int32_t *kept_seq_offsets,
                                  const int32_t *seq_offsets, int num_seqs, int rotary_dim, double base,
                                  double *out)
{
    if (rotary_dim < 0 || rotary_dim > head_dim || rotary_dim % 2) return -1;
    int64_t n_kept = kept_seq_offsets[num_seqs];
    int half = rotary_dim / 2;
    int64_t o = 0;
    for (int l = layer_begin; l < layer_end; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int h = 0; h < num_kv_heads; ++h)
                for (int b = 0; b < num_seqs; ++b)
                    for (int64_t j = kept_seq_offsets[b]; j < kept_seq_offsets[b + 1]; ++j) {
                        int64_t row = l * stride_layer + kv * stride_kv + h * stride_head +
                                      (int64_t)kept_pos[j] * stride_token;       /* in elements */
                        double delta = (double)(j - kept_seq_offsets[b]) -
                                       (double)(kept_pos[j] - seq_offsets[b]);
                        for (int i = 0; i < head_dim; ++i) {
                            double x = load_elem(src, dtype, row + i);
                            if (kv == 0 && i < rotary_dim) {
                                int f = i < half ? i : i - half;
                                double ang = delta * pow(base, -2.0 * f / rotary_dim);
                                double partner = load_elem(src, dtype, row + (i < half ? i + half : i - half));
                                x = i < half ? x * cos(ang) - partner * sin(ang)
                                             : x * cos(ang) + partner * sin(ang);
                            }
                            out[o++] = x;
                        }
                    }
    (void)n_kept;
    return 0;
}
