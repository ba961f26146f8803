// Interface between the host runtime and the tcgen05/TMEM fused kernel file.
#pragma once
#include "kvcar_internal.h"

namespace kvcar {

constexpr int TC_MAX_LAYERS = 512;

struct TcLayerCfg {
    uint8_t ok;        // this layer can run on the tensor-core kernel
    uint8_t nslot;     // operand ring depth (16 KB slots)
    uint16_t max_m;    // widest hidden layer among the layer's sources
    uint16_t max_in;   // most restored columns (needed heads x 64) of one source
    uint32_t smem;     // dynamic shared memory per CTA
};

struct TcState {
    bool available = false;
    const char *why = "not set up";
    TcLayerCfg layer[TC_MAX_LAYERS];
};

// Build the TMA descriptors into the host image of the weights buffer (at tmap_off),
// point every SourcePlan at its three descriptors and decide per layer whether the
// tensor-core kernel can run it.  Never fails hard: on any problem the state stays
// unavailable with a reason and the generic kernels run.
void tc_setup(TcState &tc, const kvcar_config &cfg, LayerPlan *plans_host, int n_layers, char *weights_dev,
              size_t tmap_off, char *weights_img, size_t pool_rows, const int *pool_width);
void tc_destroy(TcState &tc);
bool tc_layer_supported(const TcState &tc, int layer);
cudaError_t tc_launch_decode(const TcState &tc, const DecodeArgs &a, const SeqList &seqs, int layer, int n_chunks,
                             cudaStream_t st);

}  // namespace kvcar
