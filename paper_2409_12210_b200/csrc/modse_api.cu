// Host side of libmodse: argument checking, workspace carving and the order in
// which the stages of the MoDSE layer are enqueued (see include/modse.h).
#include <algorithm>
#include <cstdlib>
#include <new>
#include <vector>

#include "modse_internal.h"
#include "tc_gemm.h"

struct modse_layer {
    modse::LayerMeta meta;
    std::vector<int> h;           // hidden widths
    std::vector<int> h_desc;      // hidden widths, descending
    // record of the last forward, checked by backward
    const void *fwd_ws = nullptr;
    int fwd_tokens = -1;
    int fwd_dtype = -1;
    int fwd_saved = 0;
    int fwd_noise = 0;            // the last forward's logits carried the second term
    int last_launches = 0;
    float aux_alpha = 0.f;        // coefficient of the auxiliary load-balance loss added to the objective in backward
    int out_f32 = 0;              // bf16 layers: write y, dx and expert weight gradients as fp32
    modse::NoiseGate noise;       // second term of the router logits (borrowed device pointers)
    modse::TcPlan tc;             // device facts of the bf16 path, cached tensor maps
    int fuse = 0;                 // kFuse* bits requested for this layer
    int fwd_fuse = 0;             // bits the last forward ran with (backward follows them)
    int debug_checks = 0;         // guard blocks between workspace regions are written and checked
    // optional per-stage device timing: events [call][stage][start/stop]
    std::vector<cudaEvent_t> ev;
    std::vector<unsigned char> ev_used;   // [call][stage]
    int ev_calls_max = 0, ev_calls = 0;
};

namespace modse {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

WsLayout make_layout(const LayerMeta &m, const int *h_desc, int esz, int T, bool save)
{
    WsLayout L{};
    L.T = T;
    L.R = m.k * T;
    L.Pmax = (int)align_up((size_t)L.R + (size_t)(kRowPad - 1) * m.N, kRowPad);
    L.nblk = (T + kRouterTokB - 1) / kRouterTokB;
    L.nblk_bwd = (T + kRouterBwdTokB - 1) / kRouterBwdTokB;
    // sum_e cp_e*h_e <= T * (k largest widths) + (pad-1) * S
    size_t topk_sum = 0;
    for (int j = 0; j < m.k; ++j) topk_sum += (size_t)h_desc[j];
    L.hb = (size_t)T * topk_sum + (size_t)(kRowPad - 1) * m.S;
    size_t off = 0;
    L.n_canary = 0;
    // every region is followed by a 256-byte guard block (see kCanaryPattern)
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 256);
        if (L.n_canary < kMaxCanaries) L.canary[L.n_canary++] = off;
        off += 256;
        return o;
    };
    const size_t kT = (size_t)m.k * T, N = m.N;
    // head: status word and tile counters (64 bytes), then the router's histogram sums per super-block, which it
    // adds into: one cudaMemsetAsync zeroes both
    L.head_bytes = 64 + (size_t)((L.nblk + kSuperBlocks - 1) / kSuperBlocks) * m.k * N * 4;
    L.status = take(L.head_bytes);
    L.topk_idx = take(kT * 4);
    L.topk_gate = take(kT * 4);
    L.counts = take(N * 4);
    L.counts_slot = take((size_t)m.k * N * 4);
    L.offsets = take((N + 1) * 4);
    L.poffsets = take((N + 1) * 4);
    L.ebase = take((N + 1) * 8);
    L.row_of = take(kT * 4);
    L.token_of = take(kT * 4);
    L.prow_of = take(kT * 4);
    L.ptoken_of = take((size_t)L.Pmax * 4);
    L.pgate = take((size_t)L.Pmax * 4);
    L.block_counts = take((size_t)L.nblk * m.k * N * 4);
    L.logits = take((size_t)T * N * 4);
    L.aux_partial = take((size_t)L.nblk_bwd * N * 4);
    L.noise_u = take((size_t)T * N * 4);
    L.xp = take((size_t)L.Pmax * m.d * esz);
    L.hm = take(L.hb * esz);
    L.o = take((size_t)L.Pmax * m.d * 4);     // fp32 for every layer type
    if (save) {
        L.a_pre = take(L.hb * esz);   // fp32 path: pre-activations A, B; bf16 path: B*silu'(A) and silu(A)
        L.b_pre = take(L.hb * esz);
        L.dg = take(kT * 4);
        L.dz = take(kT * 4);
        L.du = take((size_t)T * N * 4);
        L.dgamma_partial = take((size_t)L.nblk_bwd * 4);
        L.dwr_partial = take((size_t)((T + kDwrTokB - 1) / kDwrTokB) * N * m.d * 4);
        L.dyp = take((size_t)L.Pmax * m.d * esz);
        L.da = take(L.hb * esz);
        L.db = take(L.hb * esz);
        L.dxp = take((size_t)L.Pmax * m.d * 4);   // fp32 for every layer type
        L.dg_slots = 4 * ((h_desc[0] + 255) / 256);
        L.dg_part = take((size_t)L.dg_slots * L.Pmax * 4);
    } else if (esz == 4) {
        // the fp32 path always materialises the two pre-activations
        L.a_pre = take(L.hb * esz);
        L.b_pre = take(L.hb * esz);
    }
    L.total = off;
    return L;
}

WsPtrs carve(void *ws, const WsLayout &L)
{
    unsigned char *b = static_cast<unsigned char *>(ws);
    WsPtrs p{};
    p.status = (int *)(b + L.status);
    p.topk_idx = (int *)(b + L.topk_idx);
    p.topk_gate = (float *)(b + L.topk_gate);
    p.counts = (int *)(b + L.counts);
    p.counts_slot = (int *)(b + L.counts_slot);
    p.offsets = (int *)(b + L.offsets);
    p.poffsets = (int *)(b + L.poffsets);
    p.ebase = (long long *)(b + L.ebase);
    p.row_of = (int *)(b + L.row_of);
    p.token_of = (int *)(b + L.token_of);
    p.prow_of = (int *)(b + L.prow_of);
    p.ptoken_of = (int *)(b + L.ptoken_of);
    p.pgate = (float *)(b + L.pgate);
    p.block_counts = (int *)(b + L.block_counts);
    p.super_counts = (int *)(b + L.status + 64);
    p.logits = (float *)(b + L.logits);
    p.aux_partial = (float *)(b + L.aux_partial);
    p.noise_u = (float *)(b + L.noise_u);
    p.du = (float *)(b + L.du);
    p.dgamma_partial = (float *)(b + L.dgamma_partial);
    p.dg = (float *)(b + L.dg);
    p.dz = (float *)(b + L.dz);
    p.dwr_partial = (float *)(b + L.dwr_partial);
    p.dg_part = (float *)(b + L.dg_part);
    p.xp = b + L.xp;
    p.a_pre = b + L.a_pre;
    p.b_pre = b + L.b_pre;
    p.hm = b + L.hm;
    p.o = b + L.o;
    p.dyp = b + L.dyp;
    p.da = b + L.da;
    p.db = b + L.db;
    p.dxp = b + L.dxp;
    return p;
}

static thread_local modse_status_t g_create_error = MODSE_OK;

static bool aligned16(const void *p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The bf16 tensor-core kernels tile the hidden axis in panels of 64 and the
// model axis in tiles of 128.
static bool tc_supported(const modse_layer *L)
{
    if (L->meta.d % 128 != 0) return false;
    for (int h : L->h)
        if (h % kPanel != 0) return false;
    return true;
}

}  // namespace modse

using namespace modse;

extern "C" {

modse_layer_t *modse_create(int d_model, int n_experts, const int *ffn_sizes, int top_k)
{
    g_create_error = MODSE_OK;
    if (ffn_sizes == nullptr || d_model < 8 || d_model % 8 != 0 || n_experts < 1 || n_experts > kMaxExperts ||
        top_k < 1 || top_k > n_experts) {
        g_create_error = MODSE_ERR_INVALID_ARG;
        return nullptr;
    }
    long long S = 0;
    for (int e = 0; e < n_experts; ++e) {
        if (ffn_sizes[e] < 16 || ffn_sizes[e] % 16 != 0) {
            g_create_error = MODSE_ERR_INVALID_ARG;
            return nullptr;
        }
        S += ffn_sizes[e];
    }
    if (S > (1ll << 30)) {
        g_create_error = MODSE_ERR_INVALID_ARG;
        return nullptr;
    }
    if (top_k > 2) {
        g_create_error = MODSE_ERR_UNSUPPORTED;
        return nullptr;
    }
    modse_layer *L = new (std::nothrow) modse_layer();
    if (L == nullptr) {
        g_create_error = MODSE_ERR_INVALID_ARG;
        return nullptr;
    }
    L->meta.d = d_model;
    L->meta.N = n_experts;
    L->meta.k = top_k;
    L->meta.S = (int)S;
    L->meta.hoff[0] = 0;
    for (int e = 0; e < n_experts; ++e) L->meta.hoff[e + 1] = L->meta.hoff[e] + ffn_sizes[e];
    for (int e = n_experts + 1; e <= kMaxExperts; ++e) L->meta.hoff[e] = L->meta.hoff[n_experts];
    L->h.assign(ffn_sizes, ffn_sizes + n_experts);
    L->h_desc = L->h;
    std::sort(L->h_desc.begin(), L->h_desc.end(), [](int a, int b) { return a > b; });
    const char *dbg = std::getenv("MODSE_DEBUG");
    L->debug_checks = (dbg != nullptr && dbg[0] != '\0' && dbg[0] != '0') ? 1 : 0;
    return L;
}

modse_status_t modse_last_create_error(void) { return g_create_error; }

static void drop_events(modse_layer *L)
{
    for (cudaEvent_t e : L->ev) cudaEventDestroy(e);
    L->ev.clear();
    L->ev_used.clear();
    L->ev_calls_max = L->ev_calls = 0;
}

modse_status_t modse_destroy(modse_layer_t *layer)
{
    if (layer) drop_events(layer);
    delete layer;
    return MODSE_OK;
}

int modse_check_pairs(const int *ffn_sizes, int n_experts, int *pair_sum_out)
{
    if (ffn_sizes == nullptr || n_experts < 2 || n_experts % 2 != 0) return 0;
    const int sum = ffn_sizes[0] + ffn_sizes[1];
    for (int p = 1; p < n_experts / 2; ++p)
        if (ffn_sizes[2 * p] + ffn_sizes[2 * p + 1] != sum) return 0;
    if (pair_sum_out) *pair_sum_out = sum;
    return 1;
}

const char *modse_status_string(modse_status_t s)
{
    switch (s) {
    case MODSE_OK: return "ok";
    case MODSE_ERR_INVALID_ARG: return "invalid argument";
    case MODSE_ERR_UNSUPPORTED: return "unsupported layer shape";
    case MODSE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MODSE_ERR_STATE: return "backward without a matching saved forward";
    case MODSE_ERR_CUDA: return "CUDA error";
    case MODSE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
    case MODSE_ERR_DEVICE_BOUNDS: return "a kernel met an index outside its buffers";
    }
    return "unknown status";
}

size_t modse_workspace_bytes(const modse_layer_t *layer, modse_dtype_t dtype, int n_tokens, int save_for_backward)
{
    if (layer == nullptr || n_tokens < 0 || (dtype != MODSE_F32 && dtype != MODSE_BF16)) return 0;
    if ((long long)n_tokens * layer->meta.k > (1ll << 30)) return 0;
    const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), dtype == MODSE_F32 ? 4 : 2, n_tokens,
                                   save_for_backward != 0);
    return L.total;
}

#define MODSE_CUDA(expr)                               \
    do {                                               \
        cudaError_t ce__ = (expr);                     \
        if (ce__ != cudaSuccess) return MODSE_ERR_CUDA; \
    } while (0)

// Brackets one stage with a pair of events when stage timing is on.
struct StageTimer {
    modse_layer *L;
    cudaStream_t s;
    int call;
    StageTimer(modse_layer *layer, cudaStream_t stream) : L(layer), s(stream), call(-1)
    {
        if (L->ev_calls_max > 0 && L->ev_calls < L->ev_calls_max) call = L->ev_calls++;
    }
    void mark(int stage, int which)
    {
        if (call < 0) return;
        const size_t i = ((size_t)call * MODSE_N_STAGES + stage);
        cudaEventRecord(L->ev[i * 2 + which], s);
        if (which == 1) L->ev_used[i] = 1;
    }
};
#define MODSE_STAGE(timer, stage, expr) \
    do {                                \
        (timer).mark((stage), 0);       \
        MODSE_CUDA(expr);               \
        (timer).mark((stage), 1);       \
    } while (0)

static modse_status_t check_common(const modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *w,
                                   int n_tokens, const void *workspace, size_t workspace_bytes, int save)
{
    if (layer == nullptr || w == nullptr || n_tokens < 0) return MODSE_ERR_INVALID_ARG;
    if (dtype != MODSE_F32 && dtype != MODSE_BF16) return MODSE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MODSE_OK;
    if ((long long)n_tokens * layer->meta.k > (1ll << 30)) return MODSE_ERR_INVALID_ARG;
    if (!aligned16(w->w_router) || !aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down))
        return MODSE_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MODSE_ERR_INVALID_ARG;
    if (dtype == MODSE_BF16 && !tc_supported(layer)) return MODSE_ERR_UNSUPPORTED;
    if (workspace_bytes < modse_workspace_bytes(layer, dtype, n_tokens, save)) return MODSE_ERR_WORKSPACE_TOO_SMALL;
    return MODSE_OK;
}

// Tensor maps of a call: encoded once per (workspace, x, weights, token count, direction) and kept in the layer.
static const TcMaps *cached_maps(modse_layer *layer, const LayerMeta &m, const WsLayout &L, const WsPtrs &p,
                                 const modse_weights_t *w, const void *x, const void *ws, bool backward)
{
    TcMapKey key;
    key.ws = ws; key.x = x; key.w_gate = w->w_gate; key.w_up = w->w_up; key.w_down = w->w_down;
    key.T = L.T; key.backward = backward ? 1 : 0;
    TcMaps &maps = backward ? layer->tc.maps_bwd : layer->tc.maps_fwd;
    TcMapKey &have = backward ? layer->tc.key_bwd : layer->tc.key_fwd;
    if (!(have == key)) {
        have = TcMapKey{};
        if (!tc_fill_maps(maps, m, L, p, w, x, backward)) return nullptr;
        have = key;
    }
    return &maps;
}

// Fusions that apply to a call: scatter-adding epilogues need fp32 outputs of a bf16 layer on the tensor-core path
// (two addends per element at most: top_k <= 2) and take dg from the row dot, since o is then never written.
static int effective_fuse(const modse_layer *layer, modse_dtype_t dtype, bool of32)
{
    if (dtype != MODSE_BF16 || tc_force_simt()) return 0;
    int f = layer->fuse & kFuseAll;
    if (!of32 || layer->meta.k > 2) f &= ~kFuseScatter;
    if (f & kFuseScatter) f |= kFuseDgRowdot;
    return f;
}

modse_status_t modse_forward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                             const void *x, int n_tokens, void *y, void *workspace, size_t workspace_bytes,
                             int save_for_backward, void *cuda_stream)
{
    modse_status_t st = check_common(layer, dtype, weights, n_tokens, workspace, workspace_bytes, save_for_backward);
    if (st != MODSE_OK) return st;
    if (n_tokens == 0) return MODSE_OK;
    if (!aligned16(x) || !aligned16(y)) return MODSE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const LayerMeta &m = layer->meta;
    const bool save = save_for_backward != 0;
    const WsLayout L = make_layout(m, layer->h_desc.data(), dtype == MODSE_F32 ? 4 : 2, n_tokens, save);
    const WsPtrs p = carve(workspace, L);
    int launches = 0;
    layer->fwd_ws = nullptr;
    const bool of32 = dtype == MODSE_BF16 && layer->out_f32 != 0;
    if (of32 && tc_force_simt()) return MODSE_ERR_UNSUPPORTED;
    const int fuse = effective_fuse(layer, dtype, of32);

    StageTimer tm(layer, s);
    MODSE_CUDA(cudaMemsetAsync(p.status, 0, L.head_bytes, s));   // status word, tile counters, super-block sums
    if (layer->debug_checks) MODSE_CUDA(launch_canaries(workspace, L, false, p.status, s));
    MODSE_STAGE(tm, 0, launch_router(dtype, m, x, weights->w_router, n_tokens, p, layer->noise, s, &launches));
    MODSE_STAGE(tm, 1, launch_rank(m, n_tokens, L.Pmax, p, s, &launches));
    // the grouped copy of x feeds the up/gate product (unless that gathers its rows itself) and its weight gradient
    if (!(fuse & kFuseGather) || save)
        MODSE_STAGE(tm, 2, launch_permute(dtype, m, x, n_tokens, L.Pmax, p, s, &launches));
    if (dtype == MODSE_F32 || tc_force_simt()) {
        // the bf16 cross-check path materialises both pre-activations, which only a saved forward has room for
        if (dtype == MODSE_BF16 && !save) return MODSE_ERR_UNSUPPORTED;
        SimtGemmArgs a{p.xp, weights->w_gate, p.a_pre, 0};
        tm.mark(3, 0);
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGate, m, L.Pmax, p, a, s, &launches));
        a.wgt = weights->w_up; a.out = p.b_pre;
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGate, m, L.Pmax, p, a, s, &launches));
        MODSE_CUDA(launch_swiglu_fwd(dtype, m, p, L.hb, s, &launches));
        tm.mark(3, 1);
        SimtGemmArgs b{p.hm, weights->w_down, p.o, 0};
        MODSE_STAGE(tm, 4, launch_simt_gemm(dtype, kDown, m, L.Pmax, p, b, s, &launches));
        MODSE_STAGE(tm, 5, launch_combine(dtype, m, n_tokens, L.Pmax, p, y, of32, s, &launches));
    } else {
        const TcMaps *maps = cached_maps(layer, m, L, p, weights, x, workspace, false);
        if (maps == nullptr) return MODSE_ERR_CUDA;
        MODSE_STAGE(tm, 3, tc_launch(layer->tc, TcUpGate, *maps, m, L, p, nullptr, save, false, fuse, nullptr, s, &launches));
        if (fuse & kFuseScatter) {
            // y starts at zero and every assignment's gated expert output is added into its token's row
            MODSE_STAGE(tm, 5, cudaMemsetAsync(y, 0, (size_t)n_tokens * m.d * sizeof(float), s));
            MODSE_STAGE(tm, 4, tc_launch(layer->tc, TcDown, *maps, m, L, p, nullptr, save, false, fuse,
                                         static_cast<float *>(y), s, &launches));
        } else {
            MODSE_STAGE(tm, 4, tc_launch(layer->tc, TcDown, *maps, m, L, p, nullptr, save, false, fuse, nullptr, s, &launches));
            MODSE_STAGE(tm, 5, launch_combine(dtype, m, n_tokens, L.Pmax, p, y, of32, s, &launches));
        }
    }

    layer->fwd_ws = workspace;
    layer->fwd_tokens = n_tokens;
    layer->fwd_dtype = (int)dtype;
    layer->fwd_saved = save ? 1 : 0;
    layer->fwd_noise = layer->noise.w_noise != nullptr ? 1 : 0;
    layer->fwd_fuse = fuse;
    layer->last_launches = launches;
    return MODSE_OK;
}

modse_status_t modse_backward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                              const void *x, const void *dy, int n_tokens, void *dx, const modse_wgrads_t *wgrads,
                              void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    modse_status_t st = check_common(layer, dtype, weights, n_tokens, workspace, workspace_bytes, 1);
    if (st != MODSE_OK) return st;
    if (wgrads == nullptr) return MODSE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MODSE_OK;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(wgrads->dw_router) ||
        !aligned16(wgrads->dw_gate) || !aligned16(wgrads->dw_up) || !aligned16(wgrads->dw_down))
        return MODSE_ERR_INVALID_ARG;
    if (layer->fwd_ws != workspace || layer->fwd_tokens != n_tokens || layer->fwd_dtype != (int)dtype ||
        !layer->fwd_saved)
        return MODSE_ERR_STATE;
    if ((layer->noise.w_noise != nullptr) != (layer->fwd_noise != 0)) return MODSE_ERR_STATE;
    if (layer->noise.w_noise != nullptr && (!aligned16(layer->noise.dw_noise) || layer->noise.dgamma == nullptr))
        return MODSE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const LayerMeta &m = layer->meta;
    const WsLayout L = make_layout(m, layer->h_desc.data(), dtype == MODSE_F32 ? 4 : 2, n_tokens, true);
    const WsPtrs p = carve(workspace, L);
    int launches = 0;
    const bool of32 = dtype == MODSE_BF16 && layer->out_f32 != 0;
    if (of32 && tc_force_simt()) return MODSE_ERR_UNSUPPORTED;
    // backward follows the forward it belongs to: a forward that added into y wrote no o, so dg must come from
    // the row dot; a forward with o may use either
    const int fuse = (layer->fwd_fuse & kFuseScatter) ? (of32 ? layer->fwd_fuse : -1)
                                                      : (effective_fuse(layer, dtype, of32) & ~kFuseScatter);
    if (fuse < 0) return MODSE_ERR_STATE;

    StageTimer tm(layer, s);
    MODSE_CUDA(cudaMemsetAsync(p.status + 4 + TcDownDgrad, 0, 4 * sizeof(int), s));   // tile counters of the backward products
    MODSE_STAGE(tm, 6, launch_dg_permute(dtype, m, dy, n_tokens, L.Pmax, p, !(fuse & kFuseDgRowdot), s, &launches));
    bool dx_holds_sum = false;
    if (dtype == MODSE_F32 || tc_force_simt()) {
        SimtGemmArgs a{p.dyp, weights->w_down, p.da, 0};                       // dHm into the dA buffer
        tm.mark(7, 0);
        MODSE_CUDA(launch_simt_gemm(dtype, kDownDgrad, m, L.Pmax, p, a, s, &launches));
        MODSE_CUDA(launch_swiglu_bwd(dtype, m, p, L.hb, s, &launches));
        tm.mark(7, 1);
        SimtGemmArgs w{p.dyp, p.hm, wgrads->dw_down, 0};
        MODSE_STAGE(tm, 8, launch_simt_gemm(dtype, kDownWgrad, m, L.Pmax, p, w, s, &launches));
        SimtGemmArgs g{p.da, weights->w_gate, p.dxp, 0};
        tm.mark(9, 0);
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGateDgrad, m, L.Pmax, p, g, s, &launches));
        g.act = p.db; g.wgt = weights->w_up; g.accumulate = 1;
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGateDgrad, m, L.Pmax, p, g, s, &launches));
        tm.mark(9, 1);
        SimtGemmArgs wg{p.da, p.xp, wgrads->dw_gate, 0};
        tm.mark(10, 0);
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGateWgrad, m, L.Pmax, p, wg, s, &launches));
        wg.act = p.db; wg.out = wgrads->dw_up;
        MODSE_CUDA(launch_simt_gemm(dtype, kUpGateWgrad, m, L.Pmax, p, wg, s, &launches));
        tm.mark(10, 1);
    } else {
        const TcMaps *maps = cached_maps(layer, m, L, p, weights, x, workspace, true);
        if (maps == nullptr) return MODSE_ERR_CUDA;
        MODSE_STAGE(tm, 7, tc_launch(layer->tc, TcDownDgrad, *maps, m, L, p, wgrads, true, of32, fuse, nullptr, s, &launches));
        MODSE_STAGE(tm, 8, tc_launch(layer->tc, TcDownWgrad, *maps, m, L, p, wgrads, true, of32, fuse, nullptr, s, &launches));
        if (fuse & kFuseScatter) {
            tm.mark(9, 0);
            MODSE_CUDA(cudaMemsetAsync(dx, 0, (size_t)n_tokens * m.d * sizeof(float), s));
            MODSE_CUDA(tc_launch(layer->tc, TcUpGateDgrad, *maps, m, L, p, wgrads, true, of32, fuse,
                                 static_cast<float *>(dx), s, &launches));
            tm.mark(9, 1);
            dx_holds_sum = true;
        } else {
            MODSE_STAGE(tm, 9, tc_launch(layer->tc, TcUpGateDgrad, *maps, m, L, p, wgrads, true, of32, fuse, nullptr, s, &launches));
        }
        MODSE_STAGE(tm, 10, tc_launch(layer->tc, TcUpGateWgrad, *maps, m, L, p, wgrads, true, of32, fuse, nullptr, s, &launches));
    }
    MODSE_STAGE(tm, 11, launch_router_bwd(dtype, m, x, weights->w_router, n_tokens, L.Pmax, L.nblk_bwd, p, dx, of32,
                                          dx_holds_sum, static_cast<float *>(wgrads->dw_router),
                                          layer->aux_alpha * (float)m.N / (float)n_tokens, layer->noise, s,
                                          &launches));
    layer->last_launches = launches;
    return MODSE_OK;
}

modse_status_t modse_get_routing(const modse_layer_t *layer, const void *workspace, int n_tokens,
                                 const int **topk_idx, const float **topk_gate, const int **counts,
                                 const int **counts_slot, const int **offsets, const int **row_of,
                                 const int **token_of)
{
    if (layer == nullptr || workspace == nullptr || n_tokens < 1) return MODSE_ERR_INVALID_ARG;
    if (layer->fwd_ws != workspace || layer->fwd_tokens != n_tokens) return MODSE_ERR_STATE;
    const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), layer->fwd_dtype == MODSE_F32 ? 4 : 2,
                                   n_tokens, layer->fwd_saved != 0);
    const WsPtrs p = carve(const_cast<void *>(workspace), L);
    if (topk_idx) *topk_idx = p.topk_idx;
    if (topk_gate) *topk_gate = p.topk_gate;
    if (counts) *counts = p.counts;
    if (counts_slot) *counts_slot = p.counts_slot;
    if (offsets) *offsets = p.offsets;
    if (row_of) *row_of = p.row_of;
    if (token_of) *token_of = p.token_of;
    return MODSE_OK;
}

modse_status_t modse_get_gate_grads(const modse_layer_t *layer, const void *workspace, int n_tokens,
                                    const float **dg, const float **dz)
{
    if (layer == nullptr || workspace == nullptr || n_tokens < 1) return MODSE_ERR_INVALID_ARG;
    if (layer->fwd_ws != workspace || layer->fwd_tokens != n_tokens || !layer->fwd_saved) return MODSE_ERR_STATE;
    const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), layer->fwd_dtype == MODSE_F32 ? 4 : 2,
                                   n_tokens, true);
    const WsPtrs p = carve(const_cast<void *>(workspace), L);
    if (dg) *dg = p.dg;
    if (dz) *dz = p.dz;
    return MODSE_OK;
}

modse_status_t modse_check_device_status(modse_layer_t *layer, const void *workspace, void *cuda_stream)
{
    if (layer == nullptr || workspace == nullptr) return MODSE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (layer->debug_checks && layer->fwd_ws == workspace && layer->fwd_tokens > 0) {
        // compare the guard blocks the last forward wrote; a mismatch lands in the status word
        const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), layer->fwd_dtype == MODSE_F32 ? 4 : 2,
                                       layer->fwd_tokens, layer->fwd_saved != 0);
        void *ws = const_cast<void *>(workspace);
        if (launch_canaries(ws, L, true, static_cast<int *>(ws), s) != cudaSuccess) return MODSE_ERR_CUDA;
    }
    int word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return MODSE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MODSE_ERR_CUDA;
    if (word == kDevTimeout) return MODSE_ERR_DEVICE_TIMEOUT;
    if (word == kDevBounds) return MODSE_ERR_DEVICE_BOUNDS;
    return MODSE_OK;
}

modse_status_t modse_set_debug_checks(modse_layer_t *layer, int on)
{
    if (layer == nullptr) return MODSE_ERR_INVALID_ARG;
    layer->debug_checks = on ? 1 : 0;
    return MODSE_OK;
}

modse_status_t modse_set_fusion(modse_layer_t *layer, int flags)
{
    if (layer == nullptr || (flags & ~kFuseAll) != 0) return MODSE_ERR_INVALID_ARG;
    layer->fuse = flags;
    return MODSE_OK;
}

int modse_get_fusion(const modse_layer_t *layer) { return layer ? layer->fuse : 0; }

modse_status_t modse_debug_workspace_offsets(const modse_layer_t *layer, modse_dtype_t dtype, int n_tokens,
                                             int save_for_backward, size_t *prow_of_offset, size_t *first_guard_offset,
                                             int *padded_rows)
{
    if (layer == nullptr || n_tokens < 1 || (dtype != MODSE_F32 && dtype != MODSE_BF16)) return MODSE_ERR_INVALID_ARG;
    const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), dtype == MODSE_F32 ? 4 : 2, n_tokens,
                                   save_for_backward != 0);
    if (prow_of_offset) *prow_of_offset = L.prow_of;
    if (first_guard_offset) *first_guard_offset = L.canary[1];      // the block behind topk_idx
    if (padded_rows) *padded_rows = L.Pmax;
    return MODSE_OK;
}

int modse_last_launch_count(const modse_layer_t *layer) { return layer ? layer->last_launches : 0; }

modse_status_t modse_set_aux_loss(modse_layer_t *layer, float alpha)
{
    if (layer == nullptr || !(alpha >= 0.f)) return MODSE_ERR_INVALID_ARG;
    layer->aux_alpha = alpha;
    return MODSE_OK;
}

modse_status_t modse_aux_loss(modse_layer_t *layer, const void *workspace, int n_tokens, float alpha, float *loss,
                              float *f, float *P, void *cuda_stream)
{
    if (layer == nullptr || workspace == nullptr || n_tokens < 1 || loss == nullptr) return MODSE_ERR_INVALID_ARG;
    if (layer->fwd_ws != workspace || layer->fwd_tokens != n_tokens) return MODSE_ERR_STATE;
    const WsLayout L = make_layout(layer->meta, layer->h_desc.data(), layer->fwd_dtype == MODSE_F32 ? 4 : 2,
                                   n_tokens, layer->fwd_saved != 0);
    const WsPtrs p = carve(const_cast<void *>(workspace), L);
    int launches = 0;
    MODSE_CUDA(launch_aux_loss(layer->meta, n_tokens, L.nblk_bwd, p, alpha, loss, f, P,
                               static_cast<cudaStream_t>(cuda_stream), &launches));
    layer->last_launches = launches;
    return MODSE_OK;
}

modse_status_t modse_set_noise_gate(modse_layer_t *layer, const void *w_noise, float gamma, float eps)
{
    if (layer == nullptr || !(eps >= 0.f) || !(gamma == gamma)) return MODSE_ERR_INVALID_ARG;
    if (w_noise != nullptr && !aligned16(w_noise)) return MODSE_ERR_INVALID_ARG;
    layer->noise.w_noise = w_noise;
    layer->noise.gamma = gamma;
    layer->noise.eps = eps;
    return MODSE_OK;
}

modse_status_t modse_set_noise_grads(modse_layer_t *layer, float *dw_noise, float *dgamma)
{
    if (layer == nullptr) return MODSE_ERR_INVALID_ARG;
    layer->noise.dw_noise = dw_noise;
    layer->noise.dgamma = dgamma;
    return MODSE_OK;
}

modse_status_t modse_tune_forward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                                  const void *x, int n_tokens, void *y, void *workspace, size_t workspace_bytes,
                                  int save_for_backward, void *cuda_stream)
{
    modse_status_t st = check_common(layer, dtype, weights, n_tokens, workspace, workspace_bytes, save_for_backward);
    if (st != MODSE_OK) return st;
    if (dtype != MODSE_BF16 || tc_force_simt() || n_tokens == 0) return MODSE_OK;   // one kernel shape only
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t ev[2];
    if (cudaEventCreate(&ev[0]) != cudaSuccess) return MODSE_ERR_CUDA;
    if (cudaEventCreate(&ev[1]) != cudaSuccess) { cudaEventDestroy(ev[0]); return MODSE_ERR_CUDA; }
    const int prev = layer->tc.tile_mask;
    const int base = prev >= 0 ? prev : tc_default_plan();
    const int fwd_bits = ((1 << TcUpGate) | (1 << TcDown)) * ((1 << kTcPairShift) | 1);
    // candidates: each forward product on 128-row tiles, on 256-row tiles of one CTA, or on 256-row tiles of a
    // CTA pair.  They are timed in interleaved rounds after a warm-up, so that the drift of the clocks under
    // the power limit (a burst after idle, lower clocks later) does not favour whichever candidate runs first.
    constexpr int kCand = 9;
    int masks[kCand];
    float total_ms[kCand] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    auto shape_bits = [](int shape, int kind) {
        return shape == 2 ? ((1 << (kTcPairShift + kind)) | (1 << kind)) : (shape == 1 ? (1 << kind) : 0);
    };
    for (int cand = 0; cand < kCand; ++cand)
        masks[cand] = (base & ~fwd_bits) | shape_bits(cand % 3, TcUpGate) | shape_bits(cand / 3, TcDown);
    auto run = [&](int reps) {
        for (int rep = 0; rep < reps && st == MODSE_OK; ++rep)
            st = modse_forward(layer, dtype, weights, x, n_tokens, y, workspace, workspace_bytes, save_for_backward,
                               cuda_stream);
    };
    for (int cand = 0; cand < kCand; ++cand) {      // warm-up: every candidate twice
        layer->tc.tile_mask = masks[cand];
        run(2);
    }
    for (int round = 0; round < 3 && st == MODSE_OK; ++round)
        for (int cand = 0; cand < kCand && st == MODSE_OK; ++cand) {
            layer->tc.tile_mask = masks[cand];
            float ms = 0.f;
            if (cudaEventRecord(ev[0], s) != cudaSuccess) st = MODSE_ERR_CUDA;
            run(2);
            if (st == MODSE_OK && (cudaEventRecord(ev[1], s) != cudaSuccess || cudaEventSynchronize(ev[1]) != cudaSuccess ||
                                   cudaEventElapsedTime(&ms, ev[0], ev[1]) != cudaSuccess))
                st = MODSE_ERR_CUDA;
            total_ms[cand] += ms;
        }
    int best_mask = base;
    if (st == MODSE_OK) {
        int best = 0;
        for (int cand = 1; cand < kCand; ++cand)
            if (total_ms[cand] < total_ms[best]) best = cand;
        best_mask = masks[best];
    }
    cudaEventDestroy(ev[0]);
    cudaEventDestroy(ev[1]);
    layer->tc.tile_mask = st == MODSE_OK ? best_mask : prev;
    if (st == MODSE_OK)      // leave y and the workspace as one forward under the chosen plan produces them
        st = modse_forward(layer, dtype, weights, x, n_tokens, y, workspace, workspace_bytes, save_for_backward,
                           cuda_stream);
    return st;
}

int modse_get_tile_plan(const modse_layer_t *layer) { return layer ? layer->tc.tile_mask : -1; }

modse_status_t modse_set_tile_plan(modse_layer_t *layer, int plan)
{
    if (layer == nullptr || (plan != -1 && (plan < 0 || (plan & ~kTcPlanBits) != 0))) return MODSE_ERR_INVALID_ARG;
    layer->tc.tile_mask = plan;
    return MODSE_OK;
}

modse_status_t modse_set_output_f32(modse_layer_t *layer, int on)
{
    if (layer == nullptr) return MODSE_ERR_INVALID_ARG;
    layer->out_f32 = on ? 1 : 0;
    return MODSE_OK;
}

void modse_debug_use_fma_path(int on) { tc_set_force_simt(on); }

void modse_debug_set_default_tile_plan(int plan) { tc_set_default_plan(plan); }

void modse_debug_set_dynamic_tiles(int on) { tc_set_dynamic_tiles(on); }
void modse_debug_set_epilogue_warps(int mask_128, int mask_256, int mask_pair)
{
    tc_set_epilogue_warps16(mask_128, mask_256, mask_pair);
}

void modse_debug_set_wait_limit_ms(int ms) { tc_set_wait_limit_ms(ms); }

void modse_debug_skip_tile_loads(int product, int tile) { tc_set_skip_tile(product, tile); }

const char *modse_stage_name(int stage)
{
    static const char *names[MODSE_N_STAGES] = {"router", "rank", "permute", "upgate_gemm_swiglu", "down_gemm",
                                                "combine", "dg_permute", "down_dgrad_swiglu_bwd", "down_wgrad",
                                                "upgate_dgrad", "upgate_wgrad", "router_bwd"};
    return (stage >= 0 && stage < MODSE_N_STAGES) ? names[stage] : "";
}

modse_status_t modse_stage_timing_begin(modse_layer_t *layer, int max_calls)
{
    if (layer == nullptr || max_calls < 1 || max_calls > 4096) return MODSE_ERR_INVALID_ARG;
    drop_events(layer);
    const size_t n = (size_t)max_calls * MODSE_N_STAGES * 2;
    layer->ev.reserve(n);
    for (size_t i = 0; i < n; ++i) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) {
            drop_events(layer);
            return MODSE_ERR_CUDA;
        }
        layer->ev.push_back(e);
    }
    layer->ev_used.assign((size_t)max_calls * MODSE_N_STAGES, 0);
    layer->ev_calls_max = max_calls;
    layer->ev_calls = 0;
    return MODSE_OK;
}

modse_status_t modse_stage_timing_end(modse_layer_t *layer, float *ms_out, int *calls_out)
{
    if (layer == nullptr || ms_out == nullptr || calls_out == nullptr) return MODSE_ERR_INVALID_ARG;
    const int calls = layer->ev_calls;
    modse_status_t st = MODSE_OK;
    for (int c = 0; c < calls; ++c)
        for (int sidx = 0; sidx < MODSE_N_STAGES; ++sidx) {
            const size_t i = (size_t)c * MODSE_N_STAGES + sidx;
            float ms = -1.0f;
            if (layer->ev_used[i]) {
                if (cudaEventSynchronize(layer->ev[i * 2 + 1]) != cudaSuccess ||
                    cudaEventElapsedTime(&ms, layer->ev[i * 2], layer->ev[i * 2 + 1]) != cudaSuccess) {
                    st = MODSE_ERR_CUDA;
                    ms = -1.0f;
                }
            }
            ms_out[i] = ms;
        }
    *calls_out = calls;
    drop_events(layer);
    return st;
}

}  // extern "C"
