#include "kernels.h"
#include "../../include/bigbird.h"
namespace bigbird {
int launch_attn_fwd_sm100(const FwdArgs&, const bigbird_layout&, const DeviceLayout&, DeviceScratch&, int*, cudaError_t*) {
    return BIGBIRD_EUNSUPPORTED;
}
}
