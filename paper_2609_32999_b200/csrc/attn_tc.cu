// placeholder until the tcgen05 kernel lands
#include "launch.h"
namespace tessera {
cudaError_t launch_attn_tc(const tessera_plan *, void *, void *, const void *, void *, float *, cudaStream_t, std::string *err) {
    *err = "not built";
    return cudaErrorNotSupported;
}
}  // namespace tessera
