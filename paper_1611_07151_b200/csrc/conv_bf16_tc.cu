#include "sqn_internal.h"
namespace sqn {
int conv_bf16_supported(const ConvDesc&) { return SQN_ERR_UNSUPPORTED; }
int launch_conv_bf16(const ConvDesc&, cudaStream_t) { return SQN_ERR_UNSUPPORTED; }
size_t stem_bf16_workspace_bytes(int, int, int, int) { return 0; }
int launch_stem_bf16(const ConvDesc&, void*, size_t, cudaStream_t) { return SQN_ERR_UNSUPPORTED; }
}
