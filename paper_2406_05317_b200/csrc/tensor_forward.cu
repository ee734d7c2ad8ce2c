// Tensor-core (tcgen05 / TMEM) kernels of the LoCoCo chunk step.
#include "handle.h"

namespace lococo {

bool tensor_config_supported(const lococo_config*) { return false; }
void tensor_layout_workspace(lococo_handle*, size_t*) {}
int tensor_pack_weights(lococo_handle*, const void*, cudaStream_t) { return 0; }
bool tensor_compress_supported(const lococo_handle*, const CompressParams&) { return false; }
int tensor_compress(lococo_handle*, const CompressParams&, cudaStream_t) { return -1; }
bool tensor_attention_supported(const lococo_handle*, const AttnParams&) { return false; }
int tensor_attention(lococo_handle*, const AttnParams&, cudaStream_t) { return -1; }

}  // namespace lococo
