// Internal declarations shared by the CUDA translation units of libmodse.
// Nothing here is part of the public ABI (include/modse.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "modse.h"

namespace modse {

constexpr int kMaxExperts = 256;
constexpr int kRowPad = 128;        // every expert group is padded to a multiple of this many rows
constexpr int kRouterTokB = 64;     // tokens per block in the router / rank kernels
constexpr int kSuperBlocks = 32;    // router blocks per super-block (the router also keeps histogram sums per super-block)
constexpr int kRouterBwdTokB = 128; // tokens per block in the router backward kernel
constexpr int kDwrTokB = 64;        // tokens per partial sum of dW_router = dz^T x
constexpr int kPanel = 64;          // hidden-axis panel width of the bf16 activation layout

// Device status word values (first int of the workspace).  Ints 4..9 of the same 64-byte block are the
// tile counters of the six grouped products (zeroed with it); the router's histogram sums per super-block
// (super_counts) follow the block directly and are zeroed by the same call.
enum : int { kDevOk = 0, kDevTimeout = 1, kDevBounds = 2 };

// Every workspace region is followed by a 256-byte guard block.  With the debug checks on its first 8 bytes
// hold a pattern derived from the block's index; a kernel that wrote past its region destroys it.
constexpr int kMaxCanaries = 48;
constexpr unsigned long long kCanaryPattern = 0x5EDC0DE5CA9A51E5ull;

// Layer shape, passed by value to kernels (prefix sums of the hidden widths).
struct LayerMeta {
    int d, N, k, S;
    int hoff[kMaxExperts + 1];
};

// Byte offsets of every region inside the caller's workspace.
struct WsLayout {
    int T, R, Pmax, nblk, nblk_bwd;
    size_t hb;   // element capacity of each [padded rows x h_e] activation buffer
    size_t head_bytes;   // status block + super_counts: what the start of a forward zeroes
    size_t status, topk_idx, topk_gate, counts, counts_slot, offsets, poffsets, ebase, row_of, token_of,
        prow_of, ptoken_of, pgate, block_counts, logits, aux_partial, noise_u, du, dgamma_partial, dg, dz, dwr_partial, xp, a_pre, b_pre, hm, o, dyp, da, db, dxp,
        dg_part, total;
    int dg_slots;                    // partial row dots per padded row (up to four per 256-column tile of the widest expert)
    int n_canary;
    size_t canary[kMaxCanaries];     // byte offsets of the guard blocks
};

// Pointers carved out of the workspace (device addresses).
struct WsPtrs {
    int *status, *topk_idx;
    float *topk_gate;
    int *counts, *counts_slot, *offsets, *poffsets;
    long long *ebase;
    int *row_of, *token_of, *prow_of, *ptoken_of;
    float *pgate;
    int *block_counts;
    int *super_counts;   // [ceil(nblk / kSuperBlocks)][k*N] sums of block_counts over super-blocks
    float *logits;       // [T,N] router logits (may be null: not stored)
    float *aux_partial;  // [nblk_bwd][N] partial sums of the router probabilities
    float *noise_u;      // [T,N] x W_n, kept for the backward of the second term of Eq. 2
    float *du;           // [T,N] gradient w.r.t. x W_n
    float *dgamma_partial;  // [nblk_bwd]
    float *dg, *dz, *dwr_partial;
    float *dg_part;      // [dg_slots][Pmax] partial sums of dg from the down-dgrad epilogue (fused variant)
    // xp: x in padded expert-grouped rows.  a_pre / b_pre: what the forward keeps for the SwiGLU backward -
    // the pre-activations A = xp W_gate^T, B = xp W_up^T on the fp32 path, B silu'(A) and silu(A) on the bf16
    // path.  hm: gated hidden rows g silu(A) B.  o / dxp: fp32 gated expert outputs / input gradients per row.
    // dyp: dY in group order.  da / db: gradients w.r.t. A and B.
    void *xp, *a_pre, *b_pre, *hm, *o, *dyp, *da, *db, *dxp;
};

// Second term of the router logits (Sec. 2, Eq. 2): RMSNorm(Softplus(x W_n)) over the expert
// entries, with scalar gamma.  w_noise == nullptr: the term is absent.
struct NoiseGate {
    const void *w_noise = nullptr;   // [N,d], layer dtype
    float gamma = 0.f, eps = 0.f;
    float *dw_noise = nullptr;       // [N,d] fp32
    float *dgamma = nullptr;         // one float
};

WsLayout make_layout(const LayerMeta &m, const int *h_sorted_desc, int elem_bytes, int T, bool save);
WsPtrs carve(void *ws, const WsLayout &L);

// ---- routing / permutation / elementwise stages (routing_kernels.cu) ----
cudaError_t launch_router(modse_dtype_t dt, const LayerMeta &m, const void *x, const void *w_router, int T,
                          const WsPtrs &p, const NoiseGate &ng, cudaStream_t s, int *launches);
cudaError_t launch_rank(const LayerMeta &m, int T, int Pmax, const WsPtrs &p, cudaStream_t s, int *launches);
// Every kernel that follows an index read from the routing tables checks it against Pmax (padded rows) or T
// (tokens) first; an index outside records kDevBounds in the status word and the access is skipped.
cudaError_t launch_permute(modse_dtype_t dt, const LayerMeta &m, const void *x, int T, int Pmax, const WsPtrs &p,
                           cudaStream_t s, int *launches);
cudaError_t launch_combine(modse_dtype_t dt, const LayerMeta &m, int T, int Pmax, const WsPtrs &p, void *y, bool out_f32,
                           cudaStream_t s, int *launches);
// with_dg: also dg[t,j] = <dY_t, o_row> / g from the stored fp32 expert outputs (otherwise only the permutation of dY)
cudaError_t launch_dg_permute(modse_dtype_t dt, const LayerMeta &m, const void *dy, int T, int Pmax, const WsPtrs &p,
                              bool with_dg, cudaStream_t s, int *launches);
// aux_scale = alpha * N / T of the auxiliary load-balance loss (Eq. 7), 0 when it is not part of the objective.
// dx_holds_sum: dx (fp32) already holds the sum of the token's dxp rows (scatter-adding up/gate dgrad).
cudaError_t launch_router_bwd(modse_dtype_t dt, const LayerMeta &m, const void *x, const void *w_router, int T,
                              int Pmax, int nblk_bwd, const WsPtrs &p, void *dx, bool out_f32, bool dx_holds_sum,
                              float *dw_router, float aux_scale, const NoiseGate &ng, cudaStream_t s, int *launches);
// guard blocks of the workspace: write the patterns / compare them (a mismatch records kDevBounds)
cudaError_t launch_canaries(void *ws, const WsLayout &L, bool check, int *status, cudaStream_t s);
// L_a = alpha N sum_i f_i P_i (Eq. 7-10) from the stored logits and the slot-0 histogram
cudaError_t launch_aux_loss(const LayerMeta &m, int T, int nblk_bwd, const WsPtrs &p, float alpha, float *loss,
                            float *f, float *P, cudaStream_t s, int *launches);

// ---- fp32-FMA grouped GEMMs and SwiGLU elementwise (simt_gemm.cu) ----
enum GemmKind : int {
    kUpGate = 0,      // C[cp_e, h_e]  = xp_e  . W_e^T          (W = w_gate or w_up)
    kDown = 1,        // o[cp_e, d]    = Hm_e  . W_down_e^T
    kDownDgrad = 2,   // dHm[cp_e,h_e] = dyp_e . W_down_e
    kDownWgrad = 3,   // dW_down_e[d,h_e] = dyp_e^T . Hm_e
    kUpGateDgrad = 4, // dxp[cp_e, d] (+)= dA_e . W_e
    kUpGateWgrad = 5  // dW_e[h_e, d]  = dA_e^T . xp_e
};
struct SimtGemmArgs {
    const void *act;   // activation operand in padded expert-grouped rows ([P,d]) or [rows,h_e] buffer
    const void *wgt;   // weight operand, or second activation operand for the weight-gradient kinds
    void *out;
    int accumulate;    // 1: out += product
};
cudaError_t launch_simt_gemm(modse_dtype_t dt, GemmKind kind, const LayerMeta &m, int Pmax, const WsPtrs &p,
                             const SimtGemmArgs &a, cudaStream_t s, int *launches);
cudaError_t launch_swiglu_fwd(modse_dtype_t dt, const LayerMeta &m, const WsPtrs &p, size_t hb, cudaStream_t s,
                              int *launches);
cudaError_t launch_swiglu_bwd(modse_dtype_t dt, const LayerMeta &m, const WsPtrs &p, size_t hb, cudaStream_t s,
                              int *launches);

}  // namespace modse
