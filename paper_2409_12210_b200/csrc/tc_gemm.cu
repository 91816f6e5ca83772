#include <cstdlib>
#include <cstring>

#include "tc_gemm.h"

namespace modse {

bool tc_force_simt()
{
    static int v = -1;
    if (v < 0) {
        const char *e = std::getenv("MODSE_FORCE_SIMT");
        v = (e != nullptr && std::strcmp(e, "1") == 0) ? 1 : 0;
    }
    return v == 1;
}

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
