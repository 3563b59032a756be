// Tensor-memory attention kernel for the large scale steps (placeholder translation unit:
// reports "unsupported" until the tcgen05 path is linked in).
#include "device_common.cuh"
#include "internal.h"

namespace heatkv {
struct TcState {};
int tc_create(const heatkv_config&, void*, void*, uint64_t, TcState** out) { *out = nullptr; return HEATKV_OK; }
void tc_destroy(TcState*) {}
bool tc_supported(const TcState*, const AttnParams&, int, int, bool) { return false; }
cudaError_t launch_attn_tc(TcState*, const AttnParams&, int, int, bool, cudaStream_t, int*) {
  return cudaErrorNotSupported;
}
}  // namespace heatkv
