// Launch of the K/V compaction shared by sharpv_kv_compact and the layer-by-layer entry point.
#pragma once

#include "common.cuh"

namespace sharpv {

// Validates like sharpv_kv_compact and enqueues the compaction of the planes of [layer_begin, layer_end).
// One kept list for all layers: kept_stride = count_stride = 0, the count at n_kept_ptr[0].  A list per
// layer: layer i of the range reads kept_pos + i * kept_stride and its count at n_kept_ptr[i * count_stride].
// kv_only = 0 or 1 restricts an out-of-place call to the key or to the value planes (-1: both).
sharpv_status kv_compact_launch(const void* kv_src, const sharpv_kv_layout* src_layout, void* kv_dst,
                                const sharpv_kv_layout* dst_layout, int32_t layer_begin, int32_t layer_end,
                                const int32_t* kept_pos, const int32_t* n_kept_ptr, int64_t kept_stride,
                                int64_t count_stride, int64_t capacity, int32_t* status_word, cudaStream_t stream,
                                int kv_only = -1);

}  // namespace sharpv
