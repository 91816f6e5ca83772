// modse_route_static_scratch: routing (router logits, top-k, gates, counts,
// offsets, permutation tables) for callers that cannot allocate device memory.
//
// The regular entry points take a caller-allocated workspace.  Some callers
// have nowhere to get one from: code that runs inside a memory pool it does not
// own, a plugin called from a framework's execution callback where cudaMalloc
// is forbidden (it synchronises the device and may fail mid-step), or a tool
// that only wants the routing tables of a batch.  For them the scratch of the
// router/rank kernels lives in a fixed array inside the library image.
//
// The paper has no counterpart of this entry point; it is a packaging variant
// of the router stage (Sec. 2, Eq. 2-3) with the same kernels and results.
#include "modse_internal.h"

namespace {

// Scratch held by every GPU that loads the library, until the process exits.
constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB
static __device__ __align__(256) unsigned char g_route_scratch[kStaticScratchBytes];

// Device address of g_route_scratch per device (host copy).  Valid for this process and the device's
// current context: it is looked up on the first call, so first calls from several host threads must
// be serialised by the caller, and a cudaDeviceReset invalidates it (the library is not usable
// across a reset).
constexpr int kMaxDevices = 64;
unsigned char *g_scratch_ptr[kMaxDevices];

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct ScratchLayout {
    size_t status, counts_slot_unused, poffsets, ebase, prow_of, ptoken_of, pgate, block_counts, total;
};

ScratchLayout scratch_layout(int T, int N, int k, int Pmax, int nblk)
{
    ScratchLayout L{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.status = take(64 + (size_t)((nblk + modse::kSuperBlocks - 1) / modse::kSuperBlocks) * k * N * 4);   // status, then super-block sums
    L.poffsets = take((size_t)(N + 1) * 4);
    L.ebase = take((size_t)(N + 1) * 8);
    L.prow_of = take((size_t)k * T * 4);
    L.ptoken_of = take((size_t)Pmax * 4);
    L.pgate = take((size_t)Pmax * 4);
    L.block_counts = take((size_t)nblk * k * N * 4);
    L.total = off;
    return L;
}

}  // namespace

extern "C" modse_status_t modse_route_static_scratch(modse_dtype_t dtype, int d_model, int n_experts, int top_k,
                                                     const void *x, const void *w_router, int n_tokens,
                                                     int *topk_idx, float *topk_gate, int *counts, int *counts_slot,
                                                     int *offsets, int *row_of, int *token_of, void *cuda_stream)
{
    using namespace modse;
    if (dtype != MODSE_F32 && dtype != MODSE_BF16) return MODSE_ERR_INVALID_ARG;
    if (d_model < 8 || d_model % 8 != 0 || n_experts < 1 || n_experts > kMaxExperts || top_k < 1 || top_k > n_experts ||
        n_tokens < 0)
        return MODSE_ERR_INVALID_ARG;
    if (top_k > 2) return MODSE_ERR_UNSUPPORTED;
    if (n_tokens == 0) return MODSE_OK;
    auto aligned16 = [](const void *p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
    if (!aligned16(x) || !aligned16(w_router) || topk_idx == nullptr || topk_gate == nullptr || counts == nullptr ||
        counts_slot == nullptr || offsets == nullptr || row_of == nullptr || token_of == nullptr)
        return MODSE_ERR_INVALID_ARG;

    const long long R = (long long)top_k * n_tokens;
    if (R > (1ll << 30)) return MODSE_ERR_WORKSPACE_TOO_SMALL;
    const int nblk = (n_tokens + kRouterTokB - 1) / kRouterTokB;
    const int Pmax = (int)align_up((size_t)R + (size_t)(kRowPad - 1) * n_experts, kRowPad);
    const ScratchLayout L = scratch_layout(n_tokens, n_experts, top_k, Pmax, nblk);
    // the fixed array bounds the batch: refuse what does not fit rather than overrun it
    if (L.total > kStaticScratchBytes) return MODSE_ERR_WORKSPACE_TOO_SMALL;

    // Once per device, with that device current: the device address of the array.  In host
    // code `g_route_scratch` itself is only a handle for this lookup, never a pointer a kernel may use.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MODSE_ERR_CUDA;
    if (g_scratch_ptr[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || p == nullptr) return MODSE_ERR_CUDA;
        g_scratch_ptr[dev] = static_cast<unsigned char *>(p);
    }
    unsigned char *base = g_scratch_ptr[dev];

    LayerMeta m{};
    m.d = d_model;
    m.N = n_experts;
    m.k = top_k;
    m.S = 0;                                        // widths play no part in routing

    WsPtrs p{};
    p.status = reinterpret_cast<int *>(base + L.status);
    p.poffsets = reinterpret_cast<int *>(base + L.poffsets);
    p.ebase = reinterpret_cast<long long *>(base + L.ebase);
    p.prow_of = reinterpret_cast<int *>(base + L.prow_of);
    p.ptoken_of = reinterpret_cast<int *>(base + L.ptoken_of);
    p.pgate = reinterpret_cast<float *>(base + L.pgate);
    p.block_counts = reinterpret_cast<int *>(base + L.block_counts);
    p.super_counts = reinterpret_cast<int *>(base + L.status + 64);
    p.logits = nullptr;                             // the logits themselves are not kept
    p.topk_idx = topk_idx;
    p.topk_gate = topk_gate;
    p.counts = counts;
    p.counts_slot = counts_slot;
    p.offsets = offsets;
    p.row_of = row_of;
    p.token_of = token_of;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps the previous call's bytes: the status word and the super-block sums the router adds into
    // must start at zero, every other region is fully rewritten by the two kernels before it is read
    const size_t head = 64 + (size_t)((nblk + kSuperBlocks - 1) / kSuperBlocks) * top_k * n_experts * 4;
    if (cudaMemsetAsync(p.status, 0, head, s) != cudaSuccess) return MODSE_ERR_CUDA;
    if (launch_router(dtype, m, x, w_router, n_tokens, p, NoiseGate{}, s, nullptr) != cudaSuccess) return MODSE_ERR_CUDA;
    if (launch_rank(m, n_tokens, Pmax, p, s, nullptr) != cudaSuccess) return MODSE_ERR_CUDA;
    return MODSE_OK;
}

extern "C" size_t modse_route_static_scratch_capacity(void) { return kStaticScratchBytes; }

// The status word of the last modse_route_static_scratch call on the current device lives in the
// fixed array, where modse_check_device_status (which takes a workspace) cannot reach it.
extern "C" modse_status_t modse_route_static_scratch_status(void *cuda_stream)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MODSE_ERR_CUDA;
    if (g_scratch_ptr[dev] == nullptr) return MODSE_OK;          // no call has run on this device yet
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, g_scratch_ptr[dev], sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return MODSE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MODSE_ERR_CUDA;
    if (word == modse::kDevTimeout) return MODSE_ERR_DEVICE_TIMEOUT;
    if (word == modse::kDevBounds) return MODSE_ERR_DEVICE_BOUNDS;
    return MODSE_OK;
}
