// Temporary routing of the fast-kernel entry points to the simple executors.
#include "attn_plan.cuh"
namespace ss { namespace attn {
int32_t launch_tile_items_simple(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_leaf_items_simple(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_tile_items_umma(const Params& P, cudaStream_t st, int sm_count) { return launch_tile_items_simple(P, st, sm_count); }
}}
extern "C" int32_t ss_debug_umma_tile(const void*, const void*, float*, int32_t, int32_t, int32_t, int32_t*, void*) { return SS_ERR_UNSUPPORTED; }
