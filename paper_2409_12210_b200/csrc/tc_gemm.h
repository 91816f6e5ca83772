// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMM stages of the bf16 layer.
#pragma once

#include <cuda.h>

#include "modse_internal.h"

namespace modse {

// Host-side state owned by a layer object.
struct TcPlan {
    int sm_count = 0;   // number of SMs of the device the layer last ran on
    int tile_mask = -1; // which kernel variant runs each product (layout of tc_pair_mask()); -1: the process-wide default
};

// Process-wide debugging switch: run bf16 layers through the fp32-FMA grouped
// GEMMs instead of the tensor-core kernels.
bool tc_force_simt();
void tc_set_force_simt(int on);

// Which of the six products run on the two-CTA (cta_group::2) kernel: bit k = kind k.
void tc_set_pair_mask(int mask);
int tc_pair_mask();

// The six grouped products of the layer (Sec. 3.1, Eq. 4 and its gradient).
enum TcKind : int {
    TcUpGate = 0,       // Hm = g * silu(xp Wg^T) * (xp Wu^T), optionally saving B*silu'(A) and silu(A)
    TcDown = 1,         // o = Hm Wd^T into the fp32 buffer o
    TcDownDgrad = 2,    // dHm = g * (dyp Wd), fused SwiGLU backward -> dA, dB
    TcDownWgrad = 3,    // dWd = dyp^T Hm
    TcUpGateDgrad = 4,  // dxp = dA Wg + dB Wu into the fp32 buffer dxp
    TcUpGateWgrad = 5   // dWg = dA^T xp, dWu = dB^T xp
};

// Tensor maps of every TMA-loaded buffer (bf16, 64 x 64 boxes, 128-byte swizzle), and the same tensors
// with boxes of 128 rows: where an operand's rows are contiguous (K-major operands), one 16 KB copy fills
// what two 8 KB copies would, in the same shared-memory layout, and the larger copies measured faster.
struct TcMaps {
    CUtensorMap xp, dyp, wgate, wup, wdown, hm, da, db;
    CUtensorMap xp128, dyp128, wgate128, wup128, wdown128, hm128, da128, db128;
};

bool tc_fill_maps(TcMaps &maps, const LayerMeta &m, const WsLayout &L, const WsPtrs &p, const modse_weights_t *w,
                  bool backward);
cudaError_t tc_launch(TcPlan &plan, TcKind kind, const TcMaps &maps, const LayerMeta &m, const WsPtrs &p,
                      const modse_wgrads_t *g, bool save, bool out_f32, cudaStream_t s, int *launches);

}  // namespace modse
