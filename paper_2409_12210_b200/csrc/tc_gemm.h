// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMM stages of the bf16 layer.
#pragma once

#include "modse_internal.h"

namespace modse {

// Host-side state owned by a layer object.
struct TcPlan {
    int sm_count = 0;   // number of SMs of the device the layer last ran on
};

// Process-wide debugging switch: run bf16 layers through the fp32-FMA grouped
// GEMMs instead of the tensor-core kernels.
bool tc_force_simt();
void tc_set_force_simt(int on);

// Grouped up/gate projection with fused SwiGLU, then grouped down projection
// into the fp32 buffer o (Sec. 3.1, Eq. 4, expert by expert).
modse_status_t tc_forward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                          const modse_weights_t *w, bool save, cudaStream_t s, int *launches);
// Down-projection dgrad with fused SwiGLU backward, down wgrad, up/gate dgrad
// into the fp32 buffer dxp, up/gate wgrads.
modse_status_t tc_backward(TcPlan &plan, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                           const modse_weights_t *w, const modse_wgrads_t *g, cudaStream_t s, int *launches);

}  // namespace modse
