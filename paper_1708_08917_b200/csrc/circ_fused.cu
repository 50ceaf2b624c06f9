// S4 placeholder (replaced by the fused streaming kernel).
#include "circ_common.cuh"
namespace circ {
bool fused_fc_supported(const Layer*, int) { return false; }
int launch_fused_fc(const Layer*, const void*, void*, int, cudaStream_t) {
    set_error(CIRC_ERR_UNSUPPORTED, "fused kernel not built");
    return CIRC_ERR_UNSUPPORTED;
}
}  // namespace circ
