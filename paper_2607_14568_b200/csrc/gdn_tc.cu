// Tensor-core (tcgen05) kernel for bf16 storage -- placeholder until the kernel lands.
#include "gdn_internal.h"

namespace gdn {

bool tc_supported(int, int) { return false; }
int launch_tc(const PrefillArgs&, cudaStream_t) { return GDN_ERR_UNSUPPORTED; }

}  // namespace gdn
