// GDN scan on tensor cores (placeholder until the tcgen05 kernel lands).
#include "common.cuh"
namespace lkv {
bool gdn_scan_tensor_supported(const GdnArgs &, bool) { return false; }
cudaError_t launch_gdn_scan_tensor(const GdnArgs &, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace lkv
