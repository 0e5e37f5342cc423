// tcgen05 fused attention (placeholder until the kernel lands: reports "unsupported").
#include "vd_internal.h"
namespace vd {
bool attn_tc_supported(const AttnArgs&) { return false; }
cudaError_t launch_attn_tc(const AttnArgs&, unsigned int*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace vd
