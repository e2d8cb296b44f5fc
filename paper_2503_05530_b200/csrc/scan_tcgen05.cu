// Tensor-core scan (placeholder until the tcgen05 kernel lands): reports "not available".
#include "prox_internal.h"
namespace prox {
int launch_scan_pass_tc(prox_handle *, int, cudaStream_t) { return 1; }
}  // namespace prox
