/*
 * sharpv.h -- C ABI of the SharpV pruning hot path for NVIDIA B200 (sm_100a).
 *
 * SharpV (arxiv 2511.08003) prunes a VideoLLM's visual tokens in two stages that
 * never look at attention scores:
 *   stage one (pre-LLM, Section 3.1):  per-token spatial + temporal dissimilarity
 *     scores, an adaptive keep ratio per frame, a per-frame top-k, and a gather of
 *     the kept tokens;
 *   stage two (intra-LLM, Section 3.2): each visual token's hidden state at a chosen
 *     layer is compared with its original feature by cosine similarity; degraded
 *     tokens are dropped and the K/V rows of every layer and KV head are compacted.
 *
 * Conventions shared by every entry point
 *   - Pointers marked [dev] are device memory owned by the caller; [host] are host
 *     memory.  The library allocates nothing, frees nothing and keeps no pointer
 *     after a call returns.
 *   - Every call only enqueues work on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the default stream) and returns without synchronising.
 *   - Data-dependent sizes (how many tokens survive) are written to device memory;
 *     the caller sizes outputs by a `capacity` it chooses.
 *   - The return value reports errors the host can see (bad arguments, a workspace
 *     that is too small, a failed launch).  Errors only the device can see (more
 *     survivors than `capacity`) are written to the optional [dev] `status_word`
 *     as a sharpv_status value (the largest code wins; the caller zeroes it).
 *     Kernels never trap, assert or wait without a bound.
 *   - dtype is the storage type of tokens / hidden states / K/V rows.  All
 *     reductions accumulate in fp32 from exactly widened inputs; scores, ratios and
 *     cosines are written as fp32.
 *   - Token matrices are row major with the feature axis contiguous; `ld_*` is the
 *     row stride in elements.  Base pointers and row strides must be multiples of
 *     16 bytes and d * sizeof(element) must be a multiple of 16 bytes, otherwise
 *     SHARPV_ERR_UNSUPPORTED is returned and nothing is launched.
 */
#ifndef SHARPV_H
#define SHARPV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SHARPV_OK = 0,
    SHARPV_ERR_INVALID_ARG = 1,   /* null required pointer, non-positive size, bad range */
    SHARPV_ERR_UNSUPPORTED = 2,   /* unknown dtype, misaligned pointer or stride, size over a documented limit */
    SHARPV_ERR_WORKSPACE = 3,     /* workspace smaller than the matching *_workspace_bytes() */
    SHARPV_ERR_CAPACITY = 4,      /* (status_word only) more survivors than `capacity` */
    SHARPV_ERR_CUDA = 5,          /* a CUDA runtime call or launch failed */
    SHARPV_ERR_TIMEOUT = 6,       /* (status_word only) reserved: a bounded device-side wait gave up; no kernel waits that way at present */
    SHARPV_ERR_BOUNDS = 7         /* (status_word only, libraries built with -DSHARPV_DEBUG_BOUNDS) an index that a kernel was
                                     about to gather from or scatter to lay outside its range; the access was skipped */
} sharpv_status;

/* SHARPV_U8 (any one-byte element, e.g. an fp8 K/V cache) is accepted by sharpv_kv_compact only: rows are
 * copied bit for bit, never interpreted.  Scores and cosines need SHARPV_F32 or SHARPV_BF16. */
typedef enum { SHARPV_F32 = 0, SHARPV_BF16 = 1, SHARPV_U8 = 2 } sharpv_dtype;

/* How threshold_t * f (Eq. 5, 6) becomes an integer budget.  The paper is silent;
 * FLOOR never keeps more than the computed ratio and is the default of the binding. */
typedef enum { SHARPV_ROUND_FLOOR = 0, SHARPV_ROUND_NEAREST = 1, SHARPV_ROUND_CEIL = 2 } sharpv_round;

/* Which dissimilarity the scores use (Section 3.1.1):
 * DISSIM is Eq. 1, ||v1^ - v2^||_2 = sqrt(2 - 2 cos); ONE_MINUS_COS is the
 * alternative the same section allows for the manual, fixed-threshold variant. */
typedef enum { SHARPV_DISSIM = 0, SHARPV_ONE_MINUS_COS = 1 } sharpv_dissim_kind;

const char* sharpv_status_string(sharpv_status s);
int sharpv_version(void);

/* ------------------------------------------------------------------------------------------
 * Stage one (a): importance scores and adaptive budgets.  Section 3.1.2-3.1.3, Eq. 1-6.
 *
 * tokens  [dev]  [total_frames * f, d], row stride ld_tokens: the n x f x d view of the
 *                visual token matrix V, frames of all videos packed back to back.
 * video_frame_offsets [dev] int32[num_videos + 1], ascending, [0] = 0,
 *                [num_videos] = total_frames.  The temporal term never crosses a video.
 * For every token i of frame t:
 *   S = Dissim(F_t[i], mean(F_t))                       (Eq. 2; mean over the f raw tokens, fp32)
 *   T = Dissim(F_t[i], F_{t-1}[i])                      (Eq. 3), and T := S on a video's first
 *                                                       frame (the virtual preceding frame made
 *                                                       of the frame mean, Section 3.1.3)
 *   I = T + w * S                                       (Eq. 4)
 * and for every frame  ratio_t = ||T_t||_2 / (2 sqrt(f))   (Eq. 5, 6),
 *   k_t = clamp(round_mode(ratio_t * f), min_keep, f)   evaluated in fp32.
 * A zero vector normalises to zero (v^ = v / max(||v||, 1e-12)).
 *
 * out_importance [dev] float[total_frames*f]; out_spatial, out_temporal [dev] same shape,
 * either may be NULL; out_ratio [dev] float[total_frames]; out_k [dev] int32[total_frames].
 * workspace [dev]: at least sharpv_score_frames_workspace_bytes() bytes, 256-byte aligned,
 * contents undefined before and after.  total_frames == 0 is valid and launches nothing.
 */
size_t sharpv_score_frames_workspace_bytes(int32_t total_frames, int32_t f, int32_t d);

sharpv_status sharpv_score_frames(
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens,
    int32_t num_videos, const int32_t* video_frame_offsets, int32_t total_frames,
    int32_t f, int32_t d,
    float w, sharpv_dissim_kind dissim_kind, sharpv_round round_mode, int32_t min_keep,
    float* out_importance, float* out_spatial, float* out_temporal,
    float* out_ratio, int32_t* out_k,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage one (b): per-frame top-k and gather of the kept tokens.  Section 3.1 (first paragraph)
 * and 3.1.3 (last paragraph): in every frame the highest-scoring tokens are retained, as many as
 * the frame's adaptive ratio allows.
 *
 * In frame t the k[t] tokens that come first under (importance descending, token index
 * ascending) are kept; -0 and +0 compare equal; NaN scores are not supported.  k[t] is
 * clamped to [0, f].  f <= 8192.
 * importance [dev] float[total_frames*f]; k [dev] int32[total_frames] (out_k above, or any
 * caller-chosen budgets).
 * out_kept_index [dev] int32[capacity]: global token indices t*f+i, ascending.
 * out_kept_offsets [dev] int32[total_frames+1]: exclusive scan of k; [total_frames] = count.
 * out_num_kept [dev] int32 scalar (may be NULL): the count, even when it exceeds capacity.
 * tokens / out_tokens [dev]: if out_tokens != NULL, out_tokens[j, :] = tokens[out_kept_index[j], :]
 * as a bit copy, out_tokens dense [capacity, d].  If the count exceeds capacity nothing beyond
 * capacity is written and status_word receives SHARPV_ERR_CAPACITY.
 */
size_t sharpv_select_tokens_workspace_bytes(int32_t total_frames, int32_t f);

sharpv_status sharpv_select_tokens(
    const float* importance, const int32_t* k, int32_t total_frames, int32_t f,
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t d,
    int32_t* out_kept_index, int32_t* out_kept_offsets,
    void* out_tokens, int64_t capacity, int32_t* out_num_kept,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* Manual (semi-adaptive) variant of stage one (b): keep every token whose importance is
 * strictly greater than the fixed cut K (Section 3.1.1 last sentence; K = 1.6 in Section 4.1.4).
 * Same outputs as sharpv_select_tokens; out_kept_offsets[t] is the number kept before frame t. */
sharpv_status sharpv_select_tokens_threshold(
    const float* importance, float K, int32_t total_frames, int32_t f,
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens, int32_t d,
    int32_t* out_kept_index, int32_t* out_kept_offsets,
    void* out_tokens, int64_t capacity, int32_t* out_num_kept,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage one in one call.  Section 3.1 describes Visual SharpV as one pipeline: importance scores, from
 * them the retention ratio of every frame, and the retention of each frame's highest-scoring tokens.
 * sharpv_prune_frames computes exactly what sharpv_score_frames followed by sharpv_select_tokens (with
 * the budgets out_k) computes, and writes the same outputs, but the selection runs where the frame's
 * scores are produced: the scores are not read back from memory and two launches fall away.
 * Arguments as in those two entry points; workspace of sharpv_prune_frames_workspace_bytes() bytes,
 * 256-byte aligned.  f <= 8192; frames of more than 256 tokens and rows that are not a multiple of 128
 * bytes run the two entry points one after the other inside the call.
 */
size_t sharpv_prune_frames_workspace_bytes(int32_t total_frames, int32_t f, int32_t d);

sharpv_status sharpv_prune_frames(
    const void* tokens, sharpv_dtype dtype, int64_t ld_tokens,
    int32_t num_videos, const int32_t* video_frame_offsets, int32_t total_frames,
    int32_t f, int32_t d,
    float w, sharpv_dissim_kind dissim_kind, sharpv_round round_mode, int32_t min_keep,
    float* out_importance, float* out_spatial, float* out_temporal,
    float* out_ratio, int32_t* out_k,
    int32_t* out_kept_index, int32_t* out_kept_offsets,
    void* out_tokens, int64_t capacity, int32_t* out_num_kept,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage two (a): self-calibration.  Section 3.2.3, Eq. 7, applied per visual token.
 *
 * hidden [dev] [total_seq_tokens, d]: the hidden state G_l of the chosen layer for all
 *   sequences packed back to back (Section 3.2.1: a sequence is system, visual, instruction
 *   tokens).  visual [dev] [total_visual, d]: the original visual features V fed to layer 0.
 * Sequence b owns hidden rows [seq_offsets[b], seq_offsets[b+1]).  Its visual tokens are the
 * vis_count[b] rows that start at seq_offsets[b] + vis_begin[b]; they map one to one, in
 * order, to visual rows [vis_offsets[b], vis_offsets[b] + vis_count[b]).
 * For each visual token c = cos(hidden row, visual row); the token is discarded iff c < M
 * (kept when c == M).  Every other position is kept.  Zero vectors give c = 0.
 *
 * out_cos [dev] float[total_visual] (positions no sequence maps are left untouched).
 * out_mean_cos [dev] float[num_seqs] or NULL: mean cosine over a sequence's visual tokens
 *   (the per-layer average similarity of Section 3.2.1); 0 for a sequence without any.
 * out_kept_pos [dev] int32[capacity]: kept packed positions, ascending.
 * out_kept_seq_offsets [dev] int32[num_seqs+1]: where each sequence's survivors start;
 *   [num_seqs] = total kept, even when it exceeds capacity (then SHARPV_ERR_CAPACITY is
 *   written to status_word and nothing beyond capacity is written).
 * All five table pointers are [dev] int32.  total_seq_tokens, total_visual < 2^31.
 */
size_t sharpv_kv_calibrate_prune_workspace_bytes(int64_t total_seq_tokens, int32_t num_seqs);

sharpv_status sharpv_kv_calibrate_prune(
    const void* hidden, int64_t ld_hidden, const void* visual, int64_t ld_visual,
    sharpv_dtype dtype, int32_t d,
    int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets,
    int64_t total_seq_tokens, int64_t total_visual, float M,
    float* out_cos, float* out_mean_cos,
    int32_t* out_kept_pos, int32_t* out_kept_seq_offsets, int64_t capacity,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Allocation-free variant of sharpv_kv_calibrate_prune.  (No counterpart in the paper: this is a
 * packaging of the same operation for hosts that cannot provide scratch memory.)
 *
 * Some callers have no way to hand over a workspace: a serving engine that gave all free device
 * memory to its own K/V-cache pool at start-up and can neither carve a temporary out of it nor
 * risk a cudaMalloc that fails or stalls every stream; a plug-in that only receives the tensors
 * of the operation and has no allocator handle; a process running under a fixed memory budget
 * where any late allocation is refused.  For them the keep flags and per-chunk counts live in
 * a fixed array inside the library's device image, sized for at most
 * SHARPV_NOALLOC_MAX_SEQ_TOKENS packed positions (about 260 KB, resident on every GPU that
 * loads the library until the process exits).
 *
 * Arguments, outputs and results are those of sharpv_kv_calibrate_prune without `workspace` and
 * `workspace_bytes`.  The call performs no cudaMalloc / cudaFree and calls no allocating library
 * routine.  total_seq_tokens > SHARPV_NOALLOC_MAX_SEQ_TOKENS returns SHARPV_ERR_UNSUPPORTED and
 * launches nothing.
 * The first call on each device looks up the device address of the array (one runtime query, made
 * with that device current); make that first call outside any stream capture.  All calls on a
 * device share the one array: two calls whose kernels may overlap on the GPU (different streams
 * without ordering between them) race on it and must be serialised by the caller.  The array
 * keeps the previous call's contents; each call clears the counters it accumulates into (on the
 * stream, before its kernels) and overwrites every flag before reading it, so the caller never has
 * to clear anything between calls.
 */
#define SHARPV_NOALLOC_MAX_SEQ_TOKENS 262144

sharpv_status sharpv_kv_calibrate_prune_noalloc(
    const void* hidden, int64_t ld_hidden, const void* visual, int64_t ld_visual,
    sharpv_dtype dtype, int32_t d,
    int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets,
    int64_t total_seq_tokens, int64_t total_visual, float M,
    float* out_cos, float* out_mean_cos,
    int32_t* out_kept_pos, int32_t* out_kept_seq_offsets, int64_t capacity,
    int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage two (b): K/V compaction.  Section 3.2.3: the discarded tokens' K/V is dropped so that
 * decoding only reads the visual tokens that were retained (Section 1).
 *
 * For every layer in [layer_begin, layer_end), for K and V, for every KV head:
 *     dst[j, :] = src[kept_pos[j], :]      for j < n_kept = kept_seq_offsets[num_seqs]
 * as a bit copy of head_dim elements.  Strides are in elements; the head_dim axis is
 * contiguous; every stride * sizeof(element) and head_dim * sizeof(element) must be a
 * multiple of 16 bytes; a row (head_dim elements) may be at most 16 KB.  The benchmarked layout is
 * [L][2][H][T][D_h]; a token-major cache is expressed through the strides.  kv_dst == kv_src with identical strides
 * compacts in place (kept_pos must then be strictly ascending, as sharpv_kv_calibrate_prune writes it; serving
 * stacks that cannot afford a second cache use this);
 * otherwise dst must not overlap src: the byte ranges that the first `capacity` token rows of the planes of
 * [layer_begin, layer_end) span in the two caches must be disjoint, or SHARPV_ERR_INVALID_ARG is returned and
 * nothing is launched.  Rows of dst at and beyond
 * n_kept are left untouched.  `capacity` is an upper bound on n_kept that the host knows
 * (for example total_seq_tokens) and sizes the launch; rows beyond it are not copied.
 */
typedef struct {
    int32_t num_layers, num_kv_heads, head_dim;
    sharpv_dtype dtype;
    int64_t stride_layer;   /* elements between layers */
    int64_t stride_kv;      /* elements from a layer's K block to its V block */
    int64_t stride_head;    /* elements between KV heads */
    int64_t stride_token;   /* elements between consecutive tokens */
} sharpv_kv_layout;

sharpv_status sharpv_kv_compact(
    const void* kv_src, const sharpv_kv_layout* src_layout /* [host] */,
    void* kv_dst, const sharpv_kv_layout* dst_layout /* [host] */,
    int32_t layer_begin, int32_t layer_end,
    const int32_t* kept_pos, const int32_t* kept_seq_offsets, int32_t num_seqs,
    int64_t capacity, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage two read layer by layer.  Section 3.2.3 states Eq. 7 on the hidden state of a layer l and drops
 * "the corresponding layer's" K/V; Table 1 lists the method as adaptive per layer and Section 1 calls the
 * result a hierarchical cache pruning.  All layers l in [layer_begin, layer_end) are handled by the same
 * few launches, whatever their number.  Two readings:
 *
 * SHARPV_PRUNE_PER_TOKEN  sharpv_kv_calibrate_prune on every layer's own hidden state and
 *   sharpv_kv_compact of only that layer's K and V planes with that layer's kept list, so deeper layers
 *   may keep fewer tokens than shallow ones.
 * SHARPV_PRUNE_PER_LAYER  Eq. 7 as it is printed, Discard = cos(V_l, V) < M: one decision per layer (and
 *   sequence) on the average, over the sequence's visual tokens, of the cosine between the layer's
 *   hidden state and the original feature (the per-layer similarity of Section 3.2.1).  The first layer
 *   whose average is under M loses the K/V rows of all visual tokens of that sequence, and so does
 *   every deeper layer of the range; system and instruction tokens are never dropped; a sequence
 *   without visual tokens is never cut.  The decision is taken on the device: no host synchronisation.
 *
 * hidden [dev]: the hidden states of the layers in the range, layer l at
 *   hidden + (l - layer_begin) * stride_hidden_layer elements, each [total_seq_tokens, d] with row
 *   stride ld_hidden; stride_hidden_layer * sizeof(element) must be a multiple of 16 bytes.
 * Outputs are per layer, layer l at index i = l - layer_begin:
 *   out_cos [dev] float[i * total_visual ...], out_mean_cos [dev] float[i * num_seqs ...] or NULL,
 *   out_kept_pos [dev] int32[i * capacity ...], out_kept_seq_offsets [dev] int32[i * (num_seqs + 1) ...].
 *   out_first_discard [dev] int32[num_seqs] or NULL (per-layer reading only; must be NULL otherwise): the
 *   first discarded layer of each sequence, layer_end if none.
 * kv_src / kv_dst and their layouts as in sharpv_kv_compact (kv_dst == kv_src compacts in place; both NULL:
 * decisions only, no compaction); rows of a layer's planes at and beyond that layer's kept count are left
 * untouched.  Workspace: sharpv_kv_prune_layers_workspace_bytes(total_seq_tokens, num_seqs, layer_end -
 * layer_begin) bytes.  All other arguments and the error behaviour are those of the two entry points it is
 * made of.
 */
typedef enum { SHARPV_PRUNE_PER_TOKEN = 0, SHARPV_PRUNE_PER_LAYER = 1 } sharpv_prune_mode;

size_t sharpv_kv_prune_layers_workspace_bytes(int64_t total_seq_tokens, int32_t num_seqs, int32_t num_layers);

sharpv_status sharpv_kv_prune_layers(
    const void* hidden, int64_t stride_hidden_layer, int64_t ld_hidden, const void* visual, int64_t ld_visual,
    sharpv_dtype dtype, int32_t d,
    int32_t num_seqs, const int32_t* seq_offsets, const int32_t* vis_begin,
    const int32_t* vis_count, const int32_t* vis_offsets,
    int64_t total_seq_tokens, int64_t total_visual, float M, sharpv_prune_mode mode,
    float* out_cos, float* out_mean_cos, int32_t* out_first_discard,
    int32_t* out_kept_pos, int32_t* out_kept_seq_offsets, int64_t capacity,
    const void* kv_src, const sharpv_kv_layout* src_layout /* [host] */,
    void* kv_dst, const sharpv_kv_layout* dst_layout /* [host] */,
    int32_t layer_begin, int32_t layer_end,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage two (b) with positional re-encoding.  Section 4.1.4 states that the positional embedding is
 * encoded again when Memory SharpV prunes inside the LLM; it gives no detail, so this entry point fixes
 * a reading: the cached keys carry a rotary embedding of their old position (half-split pairing:
 * dimension i pairs with i + rotary_dim/2, angle position * rope_base^(-2i/rotary_dim)).  A kept token
 * moves from p_old = kept_pos[j] - seq_offsets[b] to p_new = j - kept_seq_offsets[b] inside its
 * sequence b, so while its key row is copied it is rotated by (p_new - p_old):
 *     x1' = x1 cos - x2 sin,  x2' = x2 cos + x1 sin.
 * Angles are formed and reduced to [-pi, pi] in fp64, their sine and cosine and the rotation are taken in
 * fp32, the result is rounded to the storage type (round to nearest even); a token that does not move is
 * copied bit for bit.  Values and the dimensions at and beyond rotary_dim are bit copies; rotary_dim = 0
 * is the plain compaction.  Same arguments as sharpv_kv_compact plus seq_offsets [dev] int32[num_seqs+1]
 * (the packed sequence table of sharpv_kv_calibrate_prune), rotary_dim (even, <= head_dim,
 * (rotary_dim / 2) * sizeof(element) a multiple of 16 bytes), rope_base > 0 and a workspace of
 * sharpv_kv_compact_rope_workspace_bytes() bytes [dev] for the cos / sin table.  Out of place only;
 * SHARPV_F32 and SHARPV_BF16 caches; rows of at most 8 KB.
 */
size_t sharpv_kv_compact_rope_workspace_bytes(int64_t capacity, int32_t rotary_dim);

sharpv_status sharpv_kv_compact_rope(
    const void* kv_src, const sharpv_kv_layout* src_layout /* [host] */,
    void* kv_dst, const sharpv_kv_layout* dst_layout /* [host] */,
    int32_t layer_begin, int32_t layer_end,
    const int32_t* kept_pos, const int32_t* kept_seq_offsets, const int32_t* seq_offsets, int32_t num_seqs,
    int64_t capacity, int32_t rotary_dim, double rope_base,
    void* workspace, size_t workspace_bytes, int32_t* status_word, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SHARPV_H */
