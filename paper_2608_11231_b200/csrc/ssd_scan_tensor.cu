// SSD scan on tensor cores (placeholder until the tcgen05 kernel lands).
#include "common.cuh"
namespace lkv {
bool ssd_scan_tensor_supported(const SsdArgs &, bool) { return false; }
cudaError_t launch_ssd_scan_tensor(const SsdArgs &, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace lkv
