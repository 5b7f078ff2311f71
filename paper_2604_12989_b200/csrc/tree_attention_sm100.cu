// placeholder: replaced by the tcgen05 kernel
#include "common.cuh"
namespace ddtree {
size_t tree_attention_bf16_workspace(const AttnArgs&, const int32_t*) { return 256; }
int launch_tree_attention_bf16(const AttnArgs&, const int32_t*, void*, size_t, cudaStream_t) {
    return fail(DDTREE_ERR_UNSUPPORTED, "bf16 tree attention not built yet");
}
}  // namespace ddtree
