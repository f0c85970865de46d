#include "pconv_internal.h"
namespace pconv {
bool tiled_supported(const DeviceLayer&, int, int, int) { return false; }
cudaError_t launch_tiled(const DeviceLayer&, const void*, const float*, void*, int, int, int, bool,
                         bool, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace pconv
