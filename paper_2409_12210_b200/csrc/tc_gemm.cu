#include "tc_gemm.h"

namespace modse {

static int g_force_simt = 0;

bool tc_force_simt() { return g_force_simt != 0; }
void tc_set_force_simt(int on) { g_force_simt = on ? 1 : 0; }

modse_status_t tc_forward(TcPlan &, const LayerMeta &, const WsLayout &, const WsPtrs &, const modse_weights_t *,
                          bool, cudaStream_t, int *)
{
    return MODSE_ERR_UNSUPPORTED;
}

modse_status_t tc_backward(TcPlan &, const LayerMeta &, const WsLayout &, const WsPtrs &, const modse_weights_t *,
                           const modse_wgrads_t *, cudaStream_t, int *)
{
    return MODSE_ERR_UNSUPPORTED;
}

}  // namespace modse
