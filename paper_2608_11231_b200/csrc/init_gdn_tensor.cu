// GDN exact composition on tensor cores (placeholder until the tcgen05 kernel lands).
#include "common.cuh"
namespace lkv {
bool init_gdn_exact_tensor_supported(const InitArgs &, bool) { return false; }
cudaError_t launch_init_gdn_exact_tensor(const InitArgs &, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace lkv
