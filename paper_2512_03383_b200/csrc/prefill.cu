// Prefill kernel (M >= 64): placeholder until the tcgen05 path lands.
#include "common.cuh"
namespace uniql {
int prefill_supported(const Params&) { return 0; }
int launch_prefill(const Params&, const LaunchCfg&) { return UNIQL_ERR_UNSUPPORTED; }
}  // namespace uniql
