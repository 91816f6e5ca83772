// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMM stages of the bf16 layer.
#pragma once

#include "modse_internal.h"

namespace modse {

// Host-side cache owned by a layer object (tensor maps keyed by the buffers
// they describe).
struct TcPlan {
    int dummy = 0;
};

// True when the environment asks for the fp32-FMA cross-check path
// (MODSE_FORCE_SIMT=1); meant for debugging only.
bool tc_force_simt();

modse_status_t tc_forward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                          const modse_weights_t *w, bool save, cudaStream_t s, int *launches);
modse_status_t tc_backward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                           const modse_weights_t *w, const modse_wgrads_t *g, cudaStream_t s, int *launches);

}  // namespace modse
