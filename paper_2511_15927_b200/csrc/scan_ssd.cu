// placeholder until the tensor-core chunked scan lands
#include "dm_internal.h"
namespace dm {
bool scan_ssd_supports(const ScanArgs &) { return false; }
size_t scan_ssd_workspace_bytes(const ScanArgs &) { return 0; }
cudaError_t scan_ssd(const ScanArgs &, void *, cudaStream_t) { return cudaErrorNotSupported; }
}
