// placeholder until the tensor-core conv lands
#include "rtn_internal.cuh"
namespace rtn {
bool conv_i8_supported(const ConvArgs&) { return false; }
cudaError_t launch_conv_i8(const ConvArgs&, cudaStream_t) { return cudaErrorNotSupported; }
}
