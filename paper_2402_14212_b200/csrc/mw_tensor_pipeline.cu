#include "mw_tensor.cuh"
namespace mw {
bool tensor_supported(const mw_net*) { return false; }
void tensor_layout(mw_net*, bool, Layout& lay, size_t start) { lay.total = start; }
void tensor_destroy(mw_net*) {}
mw_status tensor_input_cotangent(mw_net*, const void* const*, const void*, const void*, void*, double*, void*, cudaStream_t) { return MW_ERR_UNSUPPORTED; }
mw_status tensor_forward_sweep(mw_net*, const void* const*, const void*, const void*, void* const*, void*, cudaStream_t) { return MW_ERR_UNSUPPORTED; }
mw_status tensor_backprop(mw_net*, const void* const*, const void*, const void*, void* const*, double*, void*, cudaStream_t) { return MW_ERR_UNSUPPORTED; }
}
