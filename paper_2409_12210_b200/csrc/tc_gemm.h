// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMM stages of the bf16 layer.
#pragma once

#include <cuda.h>

#include "modse_internal.h"

namespace modse {

// The six grouped products of the layer (Sec. 3.1, Eq. 4 and its gradient).
enum TcKind : int {
    TcUpGate = 0,       // Hm = g * silu(xp Wg^T) * (xp Wu^T), optionally saving B*silu'(A) and silu(A)
    TcDown = 1,         // o = Hm Wd^T into the fp32 buffer o
    TcDownDgrad = 2,    // dHm = g * (dyp Wd), fused SwiGLU backward -> dA, dB
    TcDownWgrad = 3,    // dWd = dyp^T Hm
    TcUpGateDgrad = 4,  // dxp = dA Wg + dB Wu into the fp32 buffer dxp
    TcUpGateWgrad = 5   // dWg = dA^T xp, dWu = dB^T xp
};

// Tile plan: one of three kernel shapes per product kind k.
//   bit 8 + k set : 256-row tiles computed by a pair of CTAs on neighbouring SMs (each stages its own 128 rows
//                   and half of the column operand; two tiles' accumulators fit, so epilogues overlap main loops);
//   else bit k set: 256-row tiles computed by one CTA (two 128-row halves that share the column operand; both
//                   accumulators belong to the tile);
//   else          : 128-row tiles, two accumulators in flight.
// Default: every product on CTA pairs; the low bits say what a product falls back to where the pair kernel does
// not apply (the row-gathering up/gate product, a device with a single SM).
constexpr int kTcPairShift = 8;
constexpr int kTcOneCtaDefault = (1 << TcDown) | (1 << TcDownWgrad) | (1 << TcUpGateDgrad) | (1 << TcUpGateWgrad);
constexpr int kTcDefaultPlan = (63 << kTcPairShift) | kTcOneCtaDefault;
constexpr int kTcPlanBits = (63 << kTcPairShift) | 63;
// Epilogue warps per CTA: bit k set = product k runs sixteen of them on its one-CTA 256-row tiles (eight
// otherwise): that shape cannot overlap its epilogue with the next main loop, so more warps shorten what is exposed.
constexpr int kTcDefaultEpi16Wide = (1 << TcUpGate) | (1 << TcDownDgrad);

// Optional fusions across the permutation (what lies either side of the permute / un-permute steps).
enum : int {
    kFuseGather = 1,    // up/gate product gathers its rows from x through the permutation (TMA gather), not from xp
    kFuseDgRowdot = 2,  // dg = rowdot(dyp Wd, Hm) / g inside the down-dgrad epilogue; o is not read in backward
    kFuseScatter = 4,   // down and up/gate dgrad add their rows straight into fp32 y / dx (k <= 2, fp32 outputs)
    kFuseAll = 7
};

// Tensor maps of every TMA-accessed buffer.
//   loads : bf16, boxes of 64 columns x 64 rows with the 128-byte swizzle, and the same tensors with boxes of
//           128 rows (where an operand's rows are contiguous one 16 KB copy fills what two 8 KB copies would);
//   xg    : x [T, d] with boxes one row high, for the row-gathering load of the fused up/gate product.
struct TcMaps {
    CUtensorMap xp, dyp, wgate, wup, wdown, hm, da, db;
    CUtensorMap xp128, dyp128, wgate128, wup128, wdown128, hm128, da128, db128;
    CUtensorMap xg;
};

// What the maps were encoded for; a call whose key matches reuses them.
struct TcMapKey {
    const void *ws = nullptr, *x = nullptr, *w_gate = nullptr, *w_up = nullptr, *w_down = nullptr;
    int T = -1, backward = -1;
    bool operator==(const TcMapKey &o) const
    {
        return ws == o.ws && x == o.x && w_gate == o.w_gate && w_up == o.w_up && w_down == o.w_down && T == o.T &&
               backward == o.backward;
    }
};

// Host-side state owned by a layer object.
struct TcPlan {
    int sm_count = 0;    // number of SMs of the device the layer last ran on
    int tile_mask = -1;  // tile plan (bit per product, see above); -1: the process-wide default
    TcMaps maps_fwd, maps_bwd;
    TcMapKey key_fwd, key_bwd;
};

// Process-wide debugging switches.
bool tc_force_simt();                 // run bf16 layers through the fp32-FMA grouped GEMMs
void tc_set_force_simt(int on);
void tc_set_default_plan(int mask);   // tile plan used by layers that have none of their own
int tc_default_plan();
void tc_set_dynamic_tiles(int on);    // 1 (default): CTAs take tiles from a shared counter; 0: tiles are dealt statically
void tc_set_wait_limit_ms(int ms);    // limit of every bounded wait inside the kernels (default 2000)
// bit per product: sixteen epilogue warps on 128-row tiles / one-CTA 256-row tiles / CTA-pair tiles
void tc_set_epilogue_warps16(int narrow_mask, int wide_mask, int pair_mask);
void tc_set_skip_tile(int kind, int tile);   // the producer of the CTA that gets `tile` of product `kind` stops there (-1: off)

bool tc_fill_maps(TcMaps &maps, const LayerMeta &m, const WsLayout &L, const WsPtrs &p, const modse_weights_t *w,
                  const void *x, bool backward);
// fuse: the kFuse* bits that apply to this product
cudaError_t tc_launch(TcPlan &plan, TcKind kind, const TcMaps &maps, const LayerMeta &m, const WsLayout &L,
                      const WsPtrs &p, const modse_wgrads_t *g, bool save, bool out_f32, int fuse, float *scatter_out,
                      cudaStream_t s, int *launches);

}  // namespace modse
