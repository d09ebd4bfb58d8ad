// Placeholder until the tcgen05/TMA kernel lands: nothing is tensor-core eligible.
#include "lordba_internal.h"

namespace lordba {
bool tc_supported(const lordba_proj &, int64_t, int) { return false; }
int launch_forward_tc(const lordba_proj *, int, int64_t, int, cudaStream_t) { return LORDBA_EUNSUPPORTED; }
}  // namespace lordba
