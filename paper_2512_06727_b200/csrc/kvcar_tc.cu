// tcgen05/TMEM fused decoder + attention kernel (bf16 storage).  Placeholder
// until the kernel lands: reports itself unavailable so the generic path runs.
#include "kvcar_tc.h"

namespace kvcar {

void tc_setup(TcState &tc, const kvcar_config &, const LayerPlan *, int, const LayerPlan *, size_t) {
    tc.available = false;
    tc.why = "tensor-core kernel not built";
}
void tc_destroy(TcState &) {}
bool tc_layer_supported(const TcState &, int) { return false; }
cudaError_t tc_launch_decode(const TcState &, const DecodeArgs &, const SeqList &, int, int, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace kvcar
