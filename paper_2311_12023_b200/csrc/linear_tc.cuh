// tcgen05 tensor-core path (large M).
#pragma once
#include "common.cuh"
namespace lq {
inline bool tc_supported(const QView&, int, int64_t, bool) { return false; }
inline size_t tc_workspace_bytes(int64_t, int64_t, int, int64_t, bool) { return 0; }
inline int tc_launch(const QView&, const void*, const void*, int, const void*, int, void*, char*, bool, cudaStream_t) { return LQLORA_ERR_UNSUPPORTED; }
}
