// Interface between the host runtime and the tcgen05/TMEM fused kernel file.
#pragma once
#include "kvcar_internal.h"

namespace kvcar {

struct TcState {
    bool available = false;
    const char *why = "not set up";
    void *impl = nullptr;  // owned by kvcar_tc.cu
};

// Build tensor maps and per-layer launch tables.  Never fails hard: on any
// problem the state stays unavailable with a reason and the generic kernels run.
void tc_setup(TcState &tc, const kvcar_config &cfg, const LayerPlan *plans_host, int n_layers,
              const LayerPlan *plans_dev, size_t pool_rows);
void tc_destroy(TcState &tc);
bool tc_layer_supported(const TcState &tc, int layer);
cudaError_t tc_launch_decode(const TcState &tc, const DecodeArgs &a, const SeqList &seqs, int layer, int n_chunks,
                             cudaStream_t st);

}  // namespace kvcar
