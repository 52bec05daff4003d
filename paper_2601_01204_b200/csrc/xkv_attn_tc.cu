// Tensor-core attention over the packed cache (placeholder until the tcgen05 kernel lands).
#include "xkv_internal.cuh"

namespace xkv {

size_t attn_tc_scratch_bytes(const xkv_params*) { return 0; }

cudaError_t launch_attn_tc(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs, float scale,
                           cudaStream_t st) {
  return launch_attn_simple(c, q, out, n, ts, hs, scale, st);  // temporary until the tcgen05 kernel lands
}

}  // namespace xkv
