// Interface of the single-kernel implementation of stage one (a) (see score_fused.cu).
#pragma once

#include "common.cuh"

namespace sharpv {

struct FusedScoreArgs {
    const void* tokens;
    sharpv_dtype dtype;
    int64_t ld_tokens;
    int num_videos;
    const int32_t* video_frame_offsets;
    int F, f, d;
    float w;
    int one_minus_cos, round_mode, min_keep;
    float *out_I, *out_S, *out_T, *out_ratio;
    int32_t* out_k;
    void* workspace;            // fused_score_workspace_bytes() bytes, 256-byte aligned (+ fused_select_workspace_bytes()
                                // behind them when select is set)
    int32_t* status_word;       // may be null
    cudaStream_t stream;
    // single-call stage one: the finaliser also selects, then one more kernel emits the kept list and the rows
    bool select;
    int32_t *out_kept_index, *out_kept_offsets, *out_num_kept;      // out_num_kept may be null
    void* out_tokens;           // may be null: indices only
    int64_t capacity;
};

// Shapes the fused kernel covers: rows that split into 128-byte column slices and frames of at most
// 256 tokens.  Everything else takes the three-kernel path.
bool fused_score_supported(sharpv_dtype dtype, int f, int d);

// Upper bound over both storage types.
size_t fused_score_workspace_bytes(int F, int f, int d);

// Staging rows of the per-frame kept lists (single-call stage one).
size_t fused_select_workspace_bytes(int F, int f);

// SHARPV_ERR_UNSUPPORTED means "could not set up (shared-memory size refused)": nothing was launched
// and the caller should take the three-kernel path.
sharpv_status fused_score_launch(const FusedScoreArgs& a);

}  // namespace sharpv
