// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMM stages of the bf16 layer.
#pragma once

#include "modse_internal.h"

namespace modse {

// Host-side cache owned by a layer object (tensor maps keyed by the buffers
// they describe).
struct TcPlan {
    int dummy = 0;
};

// Process-wide debugging switch: run bf16 layers through the fp32-FMA grouped
// GEMMs instead of the tensor-core kernels.
bool tc_force_simt();
void tc_set_force_simt(int on);

modse_status_t tc_forward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                          const modse_weights_t *w, bool save, cudaStream_t s, int *launches);
modse_status_t tc_backward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                           const modse_weights_t *w, const modse_wgrads_t *g, cudaStream_t s, int *launches);

}  // namespace modse
