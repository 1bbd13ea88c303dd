// placeholder until the tcgen05 kernel lands
#include "fc_attention.cuh"
namespace fc {
size_t attention_tc_workspace_bytes() { return 256; }
bool attention_tc_supported(const AttnGeom&, int) { return false; }
int attention_tc(fc_ctx*, cudaStream_t, const AttnGeom&, const void*, const void*, const void*, void*, void*, size_t) {
  return FC_ERR_UNIMPLEMENTED;
}
}  // namespace fc
