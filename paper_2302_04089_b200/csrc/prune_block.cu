// Placeholder translation unit; replaced by the block (attention-head) path.
#include "common.cuh"
namespace ziplm {
size_t block_workspace_bytes(int, int, int, int, int) { return 256; }
ziplm_status run_prune_blocks(const float*, const float*, int, int, int, int, float, const int*, int,
                              float*, float*, float*, int*, float*, int*, void*, size_t,
                              cudaStream_t) { return ZIPLM_ERR_UNSUPPORTED; }
}  // namespace ziplm
