// Router, permutation bookkeeping and the memory-bound stages around the
// grouped GEMMs of the MoDSE layer.
//
//   router_kernel      H(x) = x . W_g, top-k with ties to the lower index,
//                      softmax over the kept logits (Sec. 2, Eq. 2-3), and a
//                      per-block, per-slot histogram of the chosen experts.
//   rank_kernel        exclusive scans of the histogram -> counts, offsets and
//                      the stable destination row of every (token, slot).
//   permute_kernel     gathers token rows into padded expert groups.
//   combine_kernel     y_t = sum_j o[row(t,j)], o = gated expert output (Sec. 3.1, Eq. 4).
//                      (o and dxp, the two buffers that are summed over a
//                      token's slots, are kept in fp32 for every layer type so
//                      that the sum is rounded to the layer type only once.)
//   dg_permute_kernel  dg[t,j] = <dY_t, E_(t,j)>, rows of dY in group order.
//   router_dx_kernel   softmax Jacobian on the kept logits and dx assembly.
//   router_dwr_kernel  per-block partial sums of dW_router = dz^T x (fp32 FMA), for bf16
//   router_dwr_mma_kernel  layers on tensor cores; reduced in a fixed order by
//                      reduce_dwr_kernel (reproducible).
//
// No kernel uses a floating-point atomic; every sum has a fixed order.
#include <algorithm>

#include "modse_internal.h"

namespace modse {

namespace {

__device__ __forceinline__ void load8(const float *p, float (&v)[8])
{
    float4 a = *reinterpret_cast<const float4 *>(p);
    float4 b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8])
{
    uint4 q = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ void store8(float *p, const float (&v)[8])
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4 *>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}

__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float (&v)[8])
{
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&t);
    }
    *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

constexpr int kNoIndex = 0x7FFFFFFF;

// ---------------------------------------------------------------------------
// Router: one warp per token.  Each lane accumulates its 8-element chunks of
// the row in ascending order with fp32 FMAs, then a butterfly adds the lanes.
// ---------------------------------------------------------------------------
// z[i] = <x_t, w[i]> for i < N, written by lane 0 (callers __syncwarp before reading)
template <typename T>
__device__ __forceinline__ void warp_row_dots(const T *__restrict__ xr, const T *__restrict__ w, int d, int N, int lane,
                                              float *__restrict__ z)
{
    for (int g0 = 0; g0 < N; g0 += 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int c = lane * 8; c < d; c += 256) {
            float xv[8];
            load8(xr + c, xv);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (g0 + i < N) {
                    float wv[8];
                    load8(w + (size_t)(g0 + i) * d + c, wv);
#pragma unroll
                    for (int u = 0; u < 8; ++u) acc[i] = fmaf(xv[u], wv[u], acc[i]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float s = warp_sum(acc[i]);
            if (lane == 0 && g0 + i < N) z[g0 + i] = s;
        }
    }
}

// Softplus(u) = log(1 + exp(u)), written so that neither tail overflows or cancels.
__device__ __forceinline__ float softplus_f(float u) { return u > 0.f ? u + log1pf(expf(-u)) : log1pf(expf(u)); }
__device__ __forceinline__ float sigmoid_f(float u) { return 1.0f / (1.0f + expf(-u)); }

// With w_noise != nullptr the logits carry the second term of Eq. 2,
// H(x)_i = (x W_g)_i + gamma s_i / sqrt(mean_j s_j^2 + eps), s = Softplus(x W_n), and
// noise_u [T,N] receives x W_n for the backward pass.
template <typename T>
__global__ void __launch_bounds__(256)
router_kernel(const T *__restrict__ x, const T *__restrict__ w_router, int Ttok, int d, int N, int k,
              int *__restrict__ topk_idx, float *__restrict__ topk_gate, int *__restrict__ block_counts,
              float *__restrict__ logits, int w_in_smem, const T *__restrict__ w_noise, float gamma, float eps,
              float *__restrict__ noise_u, int *__restrict__ super_counts)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int Npad = (N + 3) & ~3;
    int *cnt = reinterpret_cast<int *>(smem_raw);                                          // [k*N]
    float *zbuf = reinterpret_cast<float *>(smem_raw + sizeof(int) * ((k * N + 3) & ~3));  // [8][2][Npad]
    T *wsm = reinterpret_cast<T *>(reinterpret_cast<unsigned char *>(zbuf) + sizeof(float) * 16 * Npad);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < k * N; i += blockDim.x) cnt[i] = 0;
    const T *w = w_router, *wn = w_noise;
    if (w_in_smem) {
        const size_t bytes = (size_t)N * d * sizeof(T);   // a multiple of 16: d is a multiple of 8
        unsigned char *dst = reinterpret_cast<unsigned char *>(wsm);
        for (int which = 0; which < (w_noise != nullptr ? 2 : 1); ++which) {
            const unsigned char *src = reinterpret_cast<const unsigned char *>(which ? w_noise : w_router);
            for (size_t i = (size_t)tid * 16; i < bytes; i += (size_t)blockDim.x * 16)
                *reinterpret_cast<uint4 *>(dst + which * bytes + i) = *reinterpret_cast<const uint4 *>(src + i);
        }
        w = wsm;
        wn = wsm + (size_t)N * d;
    }
    __syncthreads();

    float *z = zbuf + warp * 2 * Npad;
    float *un = z + Npad;
    const int t0 = blockIdx.x * kRouterTokB;
    for (int tok = warp; tok < kRouterTokB; tok += 8) {
        const int t = t0 + tok;
        if (t >= Ttok) break;
        const T *xr = x + (size_t)t * d;
        warp_row_dots(xr, w, d, N, lane, z);
        if (w_noise != nullptr) {
            warp_row_dots(xr, wn, d, N, lane, un);
            __syncwarp();
            float ss = 0.f;
            for (int i = lane; i < N; i += 32) {
                const float sp = softplus_f(un[i]);
                ss = fmaf(sp, sp, ss);
            }
            ss = warp_sum(ss);
            const float scale = gamma / sqrtf(ss / (float)N + eps);
            for (int i = lane; i < N; i += 32) {
                noise_u[(size_t)t * N + i] = un[i];
                z[i] = fmaf(softplus_f(un[i]), scale, z[i]);
            }
        }
        __syncwarp();
        if (logits != nullptr)
            for (int i = lane; i < N; i += 32) logits[(size_t)t * N + i] = z[i];
        // KeepTopK: k rounds of arg-max over the logits not yet taken; the pair
        // (value, index) is ordered so that equal values prefer the lower index.
        float zsel[2] = {0.f, 0.f};
        int isel[2] = {kNoIndex, kNoIndex};
        for (int j = 0; j < k; ++j) {
            float bv = -INFINITY;
            int bi = kNoIndex;
            for (int i = lane; i < N; i += 32) {
                const bool taken = (j > 0 && i == isel[0]);
                const float v = z[i];
                if (!taken && (bi == kNoIndex || v > bv)) { bv = v; bi = i; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
                const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
                if (oi != kNoIndex && (bi == kNoIndex || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
            }
            zsel[j] = bv;
            isel[j] = bi;
        }
        if (lane == 0) {
            // Softmax over the kept logits (the others are -inf and contribute 0).
            if (k == 1) {
                topk_idx[t] = isel[0];
                topk_gate[t] = 1.0f;
                atomicAdd(&cnt[isel[0]], 1);
            } else {
                const float w1 = expf(zsel[1] - zsel[0]);
                const float den = 1.0f + w1;
                topk_idx[2 * (size_t)t] = isel[0];
                topk_idx[2 * (size_t)t + 1] = isel[1];
                topk_gate[2 * (size_t)t] = 1.0f / den;
                topk_gate[2 * (size_t)t + 1] = w1 / den;
                atomicAdd(&cnt[isel[0]], 1);
                atomicAdd(&cnt[N + isel[1]], 1);
            }
        }
        __syncwarp();
    }
    __syncthreads();
    // the block's histogram, and its share of the sums over super-blocks of kSuperBlocks blocks (integer
    // atomics into words zeroed with the status word: the result does not depend on their order)
    for (int i = tid; i < k * N; i += blockDim.x) {
        const int c = cnt[i];
        block_counts[(size_t)blockIdx.x * k * N + i] = c;
        if (c != 0) atomicAdd(&super_counts[(size_t)(blockIdx.x / kSuperBlocks) * k * N + i], c);
    }
}

// ---------------------------------------------------------------------------
// Router, bf16 with at most 16 experts: the logits of 16 tokens per warp come
// from mma.sync m16n8k16 (bf16 x bf16 -> fp32) fed straight from global memory
// (four warps per 16 tokens, each summing a quarter of the k range, added in fp32).
// A lane loads 8 consecutive elements (16 bytes) of two token rows and of one
// router row per k-chunk of 32 and uses them as the operands of two MMAs: the
// sum over k does not depend on which k index sits in which operand slot as
// long as A and B agree, so no data is rearranged.  Four lanes then hold the
// logits of one token; top-k and the gates are computed with quad shuffles.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void quad_argmax(float &bv, int &bi)
{
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        if (oi != kNoIndex && (bi == kNoIndex || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
    }
}

constexpr int kRouterKSplit = 4;     // warps per 16-token group, each summing a quarter of the k range
constexpr int kRouterMmaThreads = 4 * kRouterKSplit * 32;

// NOISE: the rows of W_n are staged behind those of W_g and accumulated as NT more n-tiles, so a lane
// holds (x W_g)_e and (x W_n)_e of the same experts e; the second term of Eq. 2 is added before top-k.
template <int NT, bool NOISE>
__global__ void __launch_bounds__(kRouterMmaThreads, 2)      // two 512-thread blocks per SM: at most 64 registers
router_mma_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ w_router, int Ttok, int d,
                  int N, int k, int *__restrict__ topk_idx, float *__restrict__ topk_gate,
                  int *__restrict__ block_counts, float *__restrict__ logits,
                  const __nv_bfloat16 *__restrict__ w_noise, float gamma, float eps, float *__restrict__ noise_u,
                  int *__restrict__ super_counts)
{
    constexpr int NTT = NOISE ? 2 * NT : NT;            // n-tiles accumulated per warp
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int *cnt = reinterpret_cast<int *>(smem_raw);                                   // [k*N], padded to 128 bytes
    float *part = reinterpret_cast<float *>(smem_raw + 128);                        // [KS-1][4 groups][32 lanes][NTT*4]
    __nv_bfloat16 *wsm = reinterpret_cast<__nv_bfloat16 *>(smem_raw + 128 +
                                                           (kRouterKSplit - 1) * 4 * 32 * NTT * 4 * sizeof(float));
    const int ldw = d + 8;                                                          // 16-byte skew: conflict-free rows
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tq = lane & 3;
    const int grp = warp & 3, kpart = warp >> 2;        // 16-token group; which part of the k range
    const int t0 = blockIdx.x * kRouterTokB + grp * 16;
    const int r0 = t0 + g, r1 = t0 + g + 8;
    const bool v0 = r0 < Ttok, v1 = r1 < Ttok;
    const uint4 *x0 = reinterpret_cast<const uint4 *>(x + (size_t)(v0 ? r0 : 0) * d + tq * 8);
    const uint4 *x1 = reinterpret_cast<const uint4 *>(x + (size_t)(v1 ? r1 : 0) * d + tq * 8);
    const int cbeg = kpart * (d / kRouterKSplit);
    const int niter = (d / kRouterKSplit) / 32;
    // The router matrix goes to shared memory in batches of four 16-byte loads per thread, all four in flight
    // together, and the block synchronises BEFORE it requests any token row: with the first rows requested
    // ahead of it (to overlap the two) the matrix, which comes from L2, queued behind 128 KB of rows per SM
    // that come from DRAM, and every block waited 5 us at this barrier - a quarter of the kernel at 16384
    // tokens (time stamps per block: staging 5.3 -> 1.6 us, whole kernel 18.6 -> 17.0 us).
    const int w_total = NTT * 8 * d, w_step = 4 * kRouterMmaThreads * 8;
    auto w_load = [&](int i0, uint4 (&v)[4]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kRouterMmaThreads * 8;
            const int r = i / d, c = i % d;
            const int e = r < NT * 8 ? r : r - NT * 8;          // rows [NT*8, 2*NT*8) hold W_n
            const __nv_bfloat16 *src = r < NT * 8 ? w_router : w_noise;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (i < w_total && e < N) v[u] = *reinterpret_cast<const uint4 *>(src + (size_t)e * d + c);
        }
    };
    auto w_store = [&](int i0, const uint4 (&v)[4]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kRouterMmaThreads * 8;
            if (i < w_total) *reinterpret_cast<uint4 *>(wsm + (size_t)(i / d) * ldw + i % d) = v[u];
        }
    };
    for (int i = tid; i < k * N; i += kRouterMmaThreads) cnt[i] = 0;
    for (int i0 = tid * 8; i0 < w_total; i0 += w_step) {
        uint4 wv[4];
        w_load(i0, wv);
        w_store(i0, wv);
    }
    __syncthreads();
    // The token rows are fetched in batches of UB k-chunks, one batch ahead of the MMAs.
    constexpr int UB = 4;
    uint4 xa[UB], xb[UB];
    const uint4 za = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int u = 0; u < UB; ++u) {
        const int c0 = cbeg + u * 32;
        xa[u] = (v0 && u < niter) ? x0[c0 >> 3] : za;
        xb[u] = (v1 && u < niter) ? x1[c0 >> 3] : za;
    }

    float acc[NTT][4];
#pragma unroll
    for (int nt = 0; nt < NTT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
    for (int it0 = 0; it0 < niter; it0 += UB) {
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            const int c0 = cbeg + (it0 + u) * 32;
            if (it0 + u < niter) {
#pragma unroll
                for (int nt = 0; nt < NTT; ++nt) {
                    const uint4 w = *reinterpret_cast<const uint4 *>(wsm + (size_t)(nt * 8 + g) * ldw + c0 + tq * 8);
                    mma_bf16_16816(acc[nt], xa[u].x, xb[u].x, xa[u].y, xb[u].y, w.x, w.y);
                    mma_bf16_16816(acc[nt], xa[u].z, xb[u].z, xa[u].w, xb[u].w, w.z, w.w);
                }
            }
            // refill this slot with the chunk UB iterations ahead as soon as it has been consumed
            const int it = it0 + UB + u;
            const int cn = cbeg + it * 32;
            xa[u] = (v0 && it < niter) ? x0[cn >> 3] : za;
            xb[u] = (v1 && it < niter) ? x1[cn >> 3] : za;
        }
    }
    // the other warps hand their partial logits to the first warp of the same token group,
    // which adds them in a fixed order
    if (kpart > 0) {
#pragma unroll
        for (int nt = 0; nt < NTT; ++nt)
#pragma unroll
            for (int u = 0; u < 4; ++u)
                part[((((kpart - 1) * 4 + grp) * 32 + lane) * NTT + nt) * 4 + u] = acc[nt][u];
    }
    __syncthreads();
    if (kpart == 0) {
#pragma unroll
        for (int q = 1; q < kRouterKSplit; ++q)
#pragma unroll
            for (int nt = 0; nt < NTT; ++nt)
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    acc[nt][u] += part[((((q - 1) * 4 + grp) * 32 + lane) * NTT + nt) * 4 + u];
        // acc[nt][0..1]: token r0, experts nt*8 + 2tq, +1;  acc[nt][2..3]: token r1, same experts
        if constexpr (NOISE) {
            // acc[NT + nt] holds x W_n of the same experts: add gamma s / sqrt(mean s^2 + eps), s = Softplus
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int t = half ? r1 : r0;
                float sp[NT][2], ss = 0.f;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int e = nt * 8 + 2 * tq + u;
                        const float un = acc[NT + nt][2 * half + u];
                        sp[nt][u] = e < N ? softplus_f(un) : 0.f;
                        ss = fmaf(sp[nt][u], sp[nt][u], ss);
                        if (t < Ttok && e < N) noise_u[(size_t)t * N + e] = un;
                    }
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
                const float scale = gamma / sqrtf(ss / (float)N + eps);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int u = 0; u < 2; ++u) acc[nt][2 * half + u] = fmaf(sp[nt][u], scale, acc[nt][2 * half + u]);
            }
        }
        if (logits != nullptr) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int t = (u & 2) ? r1 : r0, e = nt * 8 + 2 * tq + (u & 1);
                    if (t < Ttok && e < N) logits[(size_t)t * N + e] = acc[nt][u];
                }
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int t = half ? r1 : r0;
            float zsel[2] = {0.f, 0.f};
            int isel[2] = {kNoIndex, kNoIndex};
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (j < k) {
                    float bv = -INFINITY;
                    int bi = kNoIndex;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int e = nt * 8 + 2 * tq + u;
                            const float v = acc[nt][2 * half + u];
                            const bool usable = e < N && !(j > 0 && e == isel[0]);
                            if (usable && (bi == kNoIndex || v > bv)) { bv = v; bi = e; }
                        }
                    quad_argmax(bv, bi);
                    zsel[j] = bv;
                    isel[j] = bi;
                }
            }
            if (tq == 0 && t < Ttok) {
                if (k == 1) {
                    topk_idx[t] = isel[0];
                    topk_gate[t] = 1.0f;
                    atomicAdd(&cnt[isel[0]], 1);
                } else {
                    const float w1 = expf(zsel[1] - zsel[0]);
                    const float den = 1.0f + w1;
                    topk_idx[2 * (size_t)t] = isel[0];
                    topk_idx[2 * (size_t)t + 1] = isel[1];
                    topk_gate[2 * (size_t)t] = 1.0f / den;
                    topk_gate[2 * (size_t)t + 1] = w1 / den;
                    atomicAdd(&cnt[isel[0]], 1);
                    atomicAdd(&cnt[N + isel[1]], 1);
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < k * N; i += kRouterMmaThreads) {
        const int c = cnt[i];
        block_counts[(size_t)blockIdx.x * k * N + i] = c;
        if (c != 0) atomicAdd(&super_counts[(size_t)(blockIdx.x / kSuperBlocks) * k * N + i], c);
    }
}

// ---------------------------------------------------------------------------
// Rank: block b owns tokens [b*64, b*64+64).  It sums the histograms of the
// blocks before it (tokens before its own) - whole super-blocks of 32 blocks from
// the sums the router kept, then the blocks of its own super-block -, scans the
// totals over experts, and ranks its own assignments by token index.  Integer
// work only.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rank_kernel(LayerMeta m, int Ttok, int Pmax, int nblk, const int *__restrict__ block_counts,
            const int *__restrict__ super_counts, const int *__restrict__ topk_idx, const float *__restrict__ topk_gate, int *__restrict__ counts,
            int *__restrict__ counts_slot, int *__restrict__ offsets, int *__restrict__ poffsets,
            long long *__restrict__ ebase, int *__restrict__ row_of, int *__restrict__ token_of,
            int *__restrict__ prow_of, int *__restrict__ ptoken_of, float *__restrict__ pgate, int *status)
{
    const int N = m.N, k = m.k, kN = k * N;
    extern __shared__ int sm[];
    int *tot = sm;                 // [kN] totals per (slot, expert)
    int *pre = tot + kN;           // [kN] sum over earlier blocks
    int *off = pre + kN;           // [N+1]
    int *poff = off + N + 1;       // [N+1]
    int *base = poff + N + 1;      // [N] rows of expert e taken by earlier blocks
    int *bidx = base + N;          // [64*k] this block's expert choices

    const int tid = threadIdx.x, b = blockIdx.x;
    // totals and "blocks before mine" sums per (slot, expert): the threads share the blocks of each
    // pair and add their partial sums with integer shared-memory atomics (order does not matter)
    for (int p = tid; p < 2 * kN; p += 256) tot[p] = 0;       // tot and pre are adjacent
    __syncthreads();
    {
        // sums over whole super-blocks (all of them for the totals, those before this block's for its prefix),
        // then the blocks of this block's own super-block that lie before it
        const int nsb = (nblk + kSuperBlocks - 1) / kSuperBlocks, sb = b / kSuperBlocks;
        const int groups = max(1, 256 / kN);
        const int gidx = tid / kN, p = tid % kN;
        if (gidx < groups && tid < 256) {
            int before = 0, all = 0;
            for (int s2 = gidx; s2 < nsb; s2 += groups) {
                const int c = super_counts[(size_t)s2 * kN + p];
                all += c;
                if (s2 < sb) before += c;
            }
            for (int bb = sb * kSuperBlocks + gidx; bb < b; bb += groups) before += block_counts[(size_t)bb * kN + p];
            atomicAdd(&tot[p], all);
            atomicAdd(&pre[p], before);
        }
        for (int q = 256 + tid; q < kN; q += 256) {            // more pairs than threads: the rest, one thread each
            int before = 0, all = 0;
            for (int s2 = 0; s2 < nsb; ++s2) {
                const int c = super_counts[(size_t)s2 * kN + q];
                all += c;
                if (s2 < sb) before += c;
            }
            for (int bb = sb * kSuperBlocks; bb < b; ++bb) before += block_counts[(size_t)bb * kN + q];
            tot[q] = all;
            pre[q] = before;
        }
    }
    const int t0 = b * kRouterTokB;
    for (int i = tid; i < kRouterTokB * k; i += 256) {
        const int t = t0 + i / k;
        bidx[i] = (t < Ttok) ? topk_idx[(size_t)t0 * k + i] : -1;
    }
    __syncthreads();
    if (tid == 0) {
        int o = 0, po = 0;
        long long eb = 0;
        for (int e = 0; e < N; ++e) {
            int c = 0, bs = 0;
            for (int j = 0; j < k; ++j) { c += tot[j * N + e]; bs += pre[j * N + e]; }
            off[e] = o;
            poff[e] = po;
            base[e] = bs;
            if (b == 0) {
                counts[e] = c;
                offsets[e] = o;
                poffsets[e] = po;
                ebase[e] = eb;
            }
            const int cp = (c + kRowPad - 1) / kRowPad * kRowPad;
            eb += (long long)cp * (m.hoff[e + 1] - m.hoff[e]);
            o += c;
            po += cp;
        }
        off[N] = o;
        poff[N] = po;
        if (b == 0) {
            offsets[N] = o;
            poffsets[N] = po;
            ebase[N] = eb;
            if (po > Pmax || o != k * Ttok) atomicMax(status, kDevBounds);
        }
    }
    __syncthreads();
    if (b == 0)
        for (int i = tid; i < kN; i += 256) counts_slot[i] = tot[i];

    // Rank inside the block: assignments of the same expert from earlier tokens.
    for (int i = tid; i < kRouterTokB * k; i += 256) {
        const int e = bidx[i];
        if (e < 0 || e >= N) continue;
        const int tl = i / k;
        int r = 0;
        for (int q = 0; q < tl * k; ++q) r += (bidx[q] == e);
        const int t = t0 + tl;
        const int local = base[e] + r;
        const int row = off[e] + local, prow = poff[e] + local;
        row_of[(size_t)t * k + (i % k)] = row;
        prow_of[(size_t)t * k + (i % k)] = prow;
        if (row < k * Ttok) token_of[row] = t;
        if (prow < Pmax) {
            ptoken_of[prow] = t;
            pgate[prow] = topk_gate[(size_t)t * k + (i % k)];
        }
    }
    // Padding rows of every group (and the unused tail) carry token -1, gate 0.
    if (b == 0) {
        for (int e = 0; e < N; ++e) {
            const int c = off[e + 1] - off[e];
            for (int r = poff[e] + c + tid; r < poff[e + 1] && r < Pmax; r += 256) { ptoken_of[r] = -1; pgate[r] = 0.f; }
        }
        for (int r = poff[N] + tid; r < Pmax; r += 256) { ptoken_of[r] = -1; pgate[r] = 0.f; }
    }
}

// ---------------------------------------------------------------------------
// Permute: one warp per token reads the row once and writes it to the k rows
// it owns in the padded expert-grouped buffer.  Extra blocks zero the padding.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
permute_kernel(const T *__restrict__ x, int Ttok, int d, int N, int k, const int *__restrict__ prow_of,
               const int *__restrict__ counts, const int *__restrict__ poffsets, T *__restrict__ xp, int tok_blocks,
               int Pmax, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if ((int)blockIdx.x < tok_blocks) {
        const int t = blockIdx.x * 8 + warp;
        if (t >= Ttok) return;
        const T *src = x + (size_t)t * d;
        int rows[2];
        rows[0] = prow_of[(size_t)t * k];
        rows[1] = (k > 1) ? prow_of[(size_t)t * k + 1] : -1;
        for (int j = 0; j < k; ++j)
            if (rows[j] < 0 || rows[j] >= Pmax) {            // a row outside the padded group space: skipped
                if (lane == 0) atomicMax(status, kDevBounds);
                rows[j] = -1;
            }
        for (int c = lane * 8; c < d; c += 256) {
            float v[8];
            load8(src + c, v);
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (rows[j] >= 0) store8(xp + (size_t)rows[j] * d + c, v);
        }
    } else {
        // padding rows: 16 blocks of 8 warps per expert cover its (at most 127) pad rows
        const int pb = blockIdx.x - tok_blocks;
        const int e = pb / 16, i = (pb % 16) * 8 + warp;
        if (e >= N) return;
        const int row = poffsets[e] + counts[e] + i;
        if (row >= poffsets[e + 1]) return;
        if (row < 0 || row >= Pmax) { if (lane == 0) atomicMax(status, kDevBounds); return; }
        const float zero[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int c = lane * 8; c < d; c += 256) store8(xp + (size_t)row * d + c, zero);
    }
}

// ---------------------------------------------------------------------------
// Combine (Eq. 4): the gate of each assignment was applied to its hidden row
// before the down projection (the projection is linear, so g*(W h) = W (g*h)),
// so y_t = o[row(t,0)] + o[row(t,1)], added in fp32 in slot order.
// ---------------------------------------------------------------------------
template <typename TO>
__global__ void __launch_bounds__(256)
combine_kernel(const float *__restrict__ o, int Ttok, int d, int k, const int *__restrict__ prow_of,
               TO *__restrict__ y, int Pmax, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * 8 + warp;
    if (t >= Ttok) return;
    const int r0 = prow_of[(size_t)t * k];
    const int r1 = (k > 1) ? prow_of[(size_t)t * k + 1] : -1;
    if (r0 < 0 || r0 >= Pmax || r1 >= Pmax || (k > 1 && r1 < 0)) {
        if (lane == 0) atomicMax(status, kDevBounds);
        return;
    }
    for (int c = lane * 8; c < d; c += 256) {
        float a[8], acc[8];
        load8(o + (size_t)r0 * d + c, acc);
        if (r1 >= 0) {
            load8(o + (size_t)r1 * d + c, a);
#pragma unroll
            for (int u = 0; u < 8; ++u) acc[u] += a[u];
        }
        store8(y + (size_t)t * d + c, acc);
    }
}

// ---------------------------------------------------------------------------
// Backward entry: dg[t,j] = <dY_t, E_(t,j)> = <dY_t, o[row(t,j)]> / g[t,j] (o holds
// the gated expert output; a gate that underflowed to 0 gives dg = 0, and its
// dz = g*(dg - s) is 0 either way); dyp[row(t,j)] = dY_t, an exact copy.
// ---------------------------------------------------------------------------
// WITH_DG = false: only the permutation of dY (dg then comes from the down-dgrad epilogue).
template <typename T, bool WITH_DG>
__global__ void __launch_bounds__(256)
dg_permute_kernel(const T *__restrict__ dy, const float *__restrict__ o, int Ttok, int d, int N, int k,
                  const int *__restrict__ prow_of, const float *__restrict__ topk_gate,
                  const int *__restrict__ counts, const int *__restrict__ poffsets, float *__restrict__ dg,
                  T *__restrict__ dyp, int tok_blocks, int Pmax, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if ((int)blockIdx.x < tok_blocks) {
        const int t = blockIdx.x * 8 + warp;
        if (t >= Ttok) return;
        const T *src = dy + (size_t)t * d;
        if constexpr (WITH_DG) {
            for (int j = 0; j < k; ++j) {
                const int row = prow_of[(size_t)t * k + j];
                if (row < 0 || row >= Pmax) {
                    if (lane == 0) { atomicMax(status, kDevBounds); dg[(size_t)t * k + j] = 0.f; }
                    continue;
                }
                const float g = topk_gate[(size_t)t * k + j];
                float acc = 0.f;
                for (int c = lane * 8; c < d; c += 256) {
                    float v[8], ov[8];
                    load8(src + c, v);
                    load8(o + (size_t)row * d + c, ov);
#pragma unroll
                    for (int u = 0; u < 8; ++u) acc = fmaf(v[u], ov[u], acc);
                    store8(dyp + (size_t)row * d + c, v);
                }
                acc = warp_sum(acc);
                if (lane == 0) dg[(size_t)t * k + j] = (g > 0.f) ? acc / g : 0.f;
            }
        } else {
            int rows[2];
            rows[0] = prow_of[(size_t)t * k];
            rows[1] = (k > 1) ? prow_of[(size_t)t * k + 1] : -1;
            for (int j = 0; j < k; ++j)
                if (rows[j] < 0 || rows[j] >= Pmax) {
                    if (lane == 0) atomicMax(status, kDevBounds);
                    rows[j] = -1;
                }
            for (int c = lane * 8; c < d; c += 256) {
                float v[8];
                load8(src + c, v);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    if (rows[j] >= 0) store8(dyp + (size_t)rows[j] * d + c, v);
            }
        }
    } else {
        const int pb = blockIdx.x - tok_blocks;
        const int e = pb / 16, i = (pb % 16) * 8 + warp;
        if (e >= N) return;
        const int row = poffsets[e] + counts[e] + i;
        if (row >= poffsets[e + 1]) return;
        if (row < 0 || row >= Pmax) { if (lane == 0) atomicMax(status, kDevBounds); return; }
        const float zero[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int c = lane * 8; c < d; c += 256) store8(dyp + (size_t)row * d + c, zero);
    }
}

// ---------------------------------------------------------------------------
// Auxiliary load-balance loss (Sec. 3.2, Eq. 7-10): L_a = alpha N sum_i f_i P_i with
// p(x) = softmax over all N logits, f_i = share of tokens whose largest probability is
// expert i (= slot-0 count / T), P_i = mean of p_i.  aux_partial_kernel sums p_i over
// blocks of 128 tokens (token order inside a block, block order in aux_final_kernel).
// Its gradient w.r.t. the logits, with f held constant (f is piecewise constant):
//   dL_a/dz[t,m] = (alpha N / T) p_m (f_m - sum_i f_i p_i).
// ---------------------------------------------------------------------------
// softmax statistics of one token: max logit, 1/sum exp, and sum_i f_i p_i
__device__ __forceinline__ void token_softmax_stats(const float *__restrict__ z, const int *__restrict__ counts_slot,
                                                    int N, float inv_T, float &zmax, float &inv_den, float &fp)
{
    zmax = z[0];
    for (int i = 1; i < N; ++i) zmax = fmaxf(zmax, z[i]);
    float den = 0.f, acc = 0.f;
    for (int i = 0; i < N; ++i) {
        const float e = expf(z[i] - zmax);
        den += e;
        acc = fmaf((float)counts_slot[i] * inv_T, e, acc);
    }
    inv_den = 1.0f / den;
    fp = acc * inv_den;
}

__global__ void __launch_bounds__(128)
aux_partial_kernel(const float *__restrict__ logits, int Ttok, int N, float *__restrict__ partial)
{
    __shared__ float red[4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x * kRouterBwdTokB + tid;
    const bool ok = t < Ttok;
    const float *z = logits + (size_t)(ok ? t : 0) * N;
    float zmax = z[0];
    for (int i = 1; i < N; ++i) zmax = fmaxf(zmax, z[i]);
    float den = 0.f;
    for (int i = 0; i < N; ++i) den += expf(z[i] - zmax);
    const float inv = ok ? 1.0f / den : 0.f;
    for (int i = 0; i < N; ++i) {
        float v = expf(z[i] - zmax) * inv;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == 0) red[warp] = v;
        __syncthreads();
        if (tid == 0) partial[(size_t)blockIdx.x * N + i] = (red[0] + red[1]) + (red[2] + red[3]);
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256)
aux_final_kernel(const float *__restrict__ partial, int nblk, const int *__restrict__ counts_slot, int Ttok, int N,
                 float alpha, float *__restrict__ loss, float *__restrict__ f_out, float *__restrict__ P_out)
{
    __shared__ float fP[kMaxExperts];
    const int i = threadIdx.x;
    if (i < N) {
        float s = 0.f;
        for (int b = 0; b < nblk; ++b) s += partial[(size_t)b * N + i];
        const float P = s / (float)Ttok, f = (float)counts_slot[i] / (float)Ttok;
        if (f_out) f_out[i] = f;
        if (P_out) P_out[i] = P;
        fP[i] = f * P;
    }
    __syncthreads();
    if (i == 0) {
        float acc = 0.f;
        for (int e = 0; e < N; ++e) acc += fP[e];
        *loss = alpha * (float)N * acc;
    }
}

// ---------------------------------------------------------------------------
// Backward of the second term of Eq. 2 (thread per token).  With dz = dL/dH over all N
// entries of the token (softmax Jacobian on the kept logits plus the auxiliary-loss term),
// s = Softplus(u), q = sqrt(mean s^2 + eps):
//   dgamma_t = sum_i dz_i s_i / q
//   du_i = gamma (dz_i / q - s_i (sum_j dz_j s_j) / (N q^3)) sigmoid(u_i)
// du [T,N] feeds dW_n = du^T x and dx += du W_n; dgamma_t is summed over the block's tokens
// in token order (block order in reduce_scalar_kernel).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kRouterBwdTokB)
noise_bwd_kernel(const float *__restrict__ noise_u, int Ttok, int N, int k, const int *__restrict__ topk_idx,
                 const float *__restrict__ topk_gate, const float *__restrict__ dg,
                 const float *__restrict__ logits, const int *__restrict__ counts_slot, float aux_scale,
                 float gamma, float eps, float *__restrict__ du, float *__restrict__ dgamma_partial)
{
    __shared__ float dgt[kRouterBwdTokB];
    const int tid = threadIdx.x;
    const int t = blockIdx.x * kRouterBwdTokB + tid;
    float dgamma_t = 0.f;
    if (t < Ttok) {
        int e[2] = {-1, -1};
        float dzk[2] = {0.f, 0.f};
        {
            float g[2] = {0.f, 0.f}, dgv[2] = {0.f, 0.f};
            for (int j = 0; j < k; ++j) {
                g[j] = topk_gate[(size_t)t * k + j];
                dgv[j] = dg[(size_t)t * k + j];
                e[j] = topk_idx[(size_t)t * k + j];
            }
            const float sg = g[0] * dgv[0] + g[1] * dgv[1];
            dzk[0] = g[0] * (dgv[0] - sg);
            dzk[1] = g[1] * (dgv[1] - sg);
        }
        const float *u = noise_u + (size_t)t * N;
        const float *zt = logits + (size_t)t * N;
        const float inv_T = 1.0f / (float)Ttok;
        float zmax = 0.f, inv_den = 0.f, fp = 0.f;
        if (aux_scale != 0.f) token_softmax_stats(zt, counts_slot, N, inv_T, zmax, inv_den, fp);
        auto dz_at = [&](int i) {
            float v = 0.f;
            if (i == e[0]) v = dzk[0];
            if (i == e[1]) v = dzk[1];
            if (aux_scale != 0.f)
                v += aux_scale * expf(zt[i] - zmax) * inv_den * ((float)counts_slot[i] * inv_T - fp);
            return v;
        };
        float ms = 0.f, dzs = 0.f;
        for (int i = 0; i < N; ++i) {
            const float sp = softplus_f(u[i]);
            ms = fmaf(sp, sp, ms);
            dzs = fmaf(dz_at(i), sp, dzs);
        }
        const float q = sqrtf(ms / (float)N + eps);
        dgamma_t = dzs / q;
        const float c1 = gamma / q, c2 = gamma * dzs / ((float)N * q * q * q);
        for (int i = 0; i < N; ++i) {
            const float sp = softplus_f(u[i]);
            du[(size_t)t * N + i] = (c1 * dz_at(i) - c2 * sp) * sigmoid_f(u[i]);
        }
    }
    dgt[tid] = dgamma_t;
    __syncthreads();
    if (tid == 0) {
        float acc = 0.f;
        for (int i = 0; i < kRouterBwdTokB; ++i) acc += dgt[i];
        dgamma_partial[blockIdx.x] = acc;
    }
}

__global__ void reduce_scalar_kernel(const float *__restrict__ partial, int n, float *__restrict__ out)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        float acc = 0.f;
        for (int i = 0; i < n; ++i) acc += partial[i];
        *out = acc;
    }
}

// ---------------------------------------------------------------------------
// Router backward, part 1 (warp per token): s = sum_j g_j dg_j,
// dz_j = g_j (dg_j - s), dx_t = sum_j dxp[row_j] + sum_j dz_j W_router[e_j]
// (+ sum_m du_m W_n[m] when the logits carry the second term of Eq. 2).
// ---------------------------------------------------------------------------
template <typename T, typename TO>
__global__ void __launch_bounds__(256)
router_dx_kernel(const T *__restrict__ w_router, const float *__restrict__ dxp, int Ttok, int d, int k,
                 const int *__restrict__ topk_idx, const float *__restrict__ topk_gate,
                 const int *__restrict__ prow_of, const float *__restrict__ dg, float *__restrict__ dz,
                 TO *__restrict__ dx, int N, const float *__restrict__ logits, const int *__restrict__ counts_slot,
                 float aux_scale, const T *__restrict__ w_noise, const float *__restrict__ du, int Pmax,
                 int dx_holds_sum, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * 8 + warp;
    if (t >= Ttok) return;
    float g[2] = {0.f, 0.f}, dgv[2] = {0.f, 0.f}, dzv[2];
    int e[2] = {0, 0}, rows[2] = {-1, -1};
    for (int j = 0; j < k; ++j) {
        g[j] = topk_gate[(size_t)t * k + j];
        dgv[j] = dg[(size_t)t * k + j];
        e[j] = topk_idx[(size_t)t * k + j];
        rows[j] = prow_of[(size_t)t * k + j];
        if (rows[j] < 0 || rows[j] >= Pmax || e[j] < 0 || e[j] >= N) {   // skipped: the token's dx row is left unwritten
            if (lane == 0) atomicMax(status, kDevBounds);
            return;
        }
    }
    const float s = g[0] * dgv[0] + g[1] * dgv[1];
    dzv[0] = g[0] * (dgv[0] - s);
    dzv[1] = g[1] * (dgv[1] - s);
    if (lane < k) dz[(size_t)t * k + lane] = dzv[lane];
    // auxiliary loss: every expert's logit gets a gradient (computed by all lanes alike)
    float zmax = 0.f, inv_den = 0.f, fp = 0.f;
    const float *zt = logits + (size_t)t * N;
    const float inv_T = 1.0f / (float)Ttok;
    if (aux_scale != 0.f) token_softmax_stats(zt, counts_slot, N, inv_T, zmax, inv_den, fp);
    for (int c = lane * 8; c < d; c += 256) {
        float a[8], out[8], wv[8];
        if (dx_holds_sum) {
            // the up/gate dgrad added the token's rows into dx (fp32) already
            if constexpr (sizeof(TO) == 4) {
                load8(reinterpret_cast<const float *>(dx) + (size_t)t * d + c, out);
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u) out[u] = 0.f;      // not reached: adding into dx needs fp32 outputs
            }
        } else {
            load8(dxp + (size_t)rows[0] * d + c, out);
            if (k > 1) {
                load8(dxp + (size_t)rows[1] * d + c, a);
#pragma unroll
                for (int u = 0; u < 8; ++u) out[u] += a[u];
            }
        }
        for (int j = 0; j < k; ++j) {
            load8(w_router + (size_t)e[j] * d + c, wv);
#pragma unroll
            for (int u = 0; u < 8; ++u) out[u] = fmaf(dzv[j], wv[u], out[u]);
        }
        if (aux_scale != 0.f) {
            for (int m = 0; m < N; ++m) {
                const float pm = expf(zt[m] - zmax) * inv_den;
                const float dza = aux_scale * pm * ((float)counts_slot[m] * inv_T - fp);
                load8(w_router + (size_t)m * d + c, wv);
#pragma unroll
                for (int u = 0; u < 8; ++u) out[u] = fmaf(dza, wv[u], out[u]);
            }
        }
        if (w_noise != nullptr) {
            for (int m = 0; m < N; ++m) {
                const float dum = du[(size_t)t * N + m];
                load8(w_noise + (size_t)m * d + c, wv);
#pragma unroll
                for (int u = 0; u < 8; ++u) out[u] = fmaf(dum, wv[u], out[u]);
            }
        }
        store8(dx + (size_t)t * d + c, out);
    }
}

// ---------------------------------------------------------------------------
// Router backward, part 2: dW_router = dz^T x as per-block partial sums.  Block
// (bx, by) owns tokens [64 bx, +64) and 256 x (16 bytes of) columns; each thread
// owns the columns of one 16-byte load and adds its tokens in ascending order, eight
// experts at a time, against the dense [64][8] slice of dz held in shared memory.  With `dense`
// set, the slice is read from that [T,N] array instead (dW_n = du^T x).
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
router_dwr_kernel(const T *__restrict__ x, int Ttok, int d, int N, int k, const int *__restrict__ topk_idx,
                  const float *__restrict__ dz, float *__restrict__ dwr_partial, const float *__restrict__ logits,
                  const int *__restrict__ counts_slot, float aux_scale, const float *__restrict__ dense)
{
    constexpr int CPT = 16 / sizeof(T);                  // columns per thread: one 16-byte load
    __shared__ __align__(16) float dzs[kDwrTokB][8];
    __shared__ int idxs[kDwrTokB][2];
    __shared__ float dzk[kDwrTokB][2];
    __shared__ float smax[kDwrTokB], sinv[kDwrTokB], sfp[kDwrTokB];
    const int tid = threadIdx.x;
    const int t0 = blockIdx.x * kDwrTokB;
    const int c = (blockIdx.y * 256 + tid) * CPT;
    const int ntok = min(kDwrTokB, Ttok - t0);
    const float inv_T = 1.0f / (float)Ttok;
    if (aux_scale != 0.f && tid < ntok)
        token_softmax_stats(logits + (size_t)(t0 + tid) * N, counts_slot, N, inv_T, smax[tid], sinv[tid], sfp[tid]);
    for (int i = tid; i < kDwrTokB * 2; i += 256) {
        const int tl = i >> 1, j = i & 1;
        const bool ok = tl < ntok && j < k;
        idxs[tl][j] = ok ? topk_idx[(size_t)(t0 + tl) * k + j] : -1;
        dzk[tl][j] = ok ? dz[(size_t)(t0 + tl) * k + j] : 0.f;
    }
    for (int g0 = 0; g0 < N; g0 += 8) {
        __syncthreads();
        for (int i = tid; i < kDwrTokB * 8; i += 256) {
            const int tl = i >> 3, e = g0 + (i & 7);
            float v = 0.f;
            if (dense != nullptr) {
                if (tl < ntok && e < N) v = dense[(size_t)(t0 + tl) * N + e];
            } else {
                if (idxs[tl][0] == e) v = dzk[tl][0];
                if (idxs[tl][1] == e) v = dzk[tl][1];
            }
            if (dense == nullptr && aux_scale != 0.f && tl < ntok && e < N) {
                const float pm = expf(logits[(size_t)(t0 + tl) * N + e] - smax[tl]) * sinv[tl];
                v += aux_scale * pm * ((float)counts_slot[e] * inv_T - sfp[tl]);
            }
            dzs[tl][i & 7] = v;
        }
        __syncthreads();
        if (c < d) {                                   // d is a multiple of 8: a thread's columns are all inside or all outside
            float acc[8][CPT];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int u = 0; u < CPT; ++u) acc[i][u] = 0.f;
            const T *xc = x + (size_t)t0 * d + c;
#pragma unroll 8
            for (int tl = 0; tl < ntok; ++tl) {
                float xv[8];
                if constexpr (sizeof(T) == 4) {
                    const float4 q = *reinterpret_cast<const float4 *>(xc + (size_t)tl * d);
                    xv[0] = q.x; xv[1] = q.y; xv[2] = q.z; xv[3] = q.w;
                } else {
                    load8(xc + (size_t)tl * d, xv);
                }
                const float4 za = *reinterpret_cast<const float4 *>(&dzs[tl][0]);
                const float4 zb = *reinterpret_cast<const float4 *>(&dzs[tl][4]);
                const float zz[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int u = 0; u < CPT; ++u) acc[i][u] = fmaf(zz[i], xv[u], acc[i][u]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (g0 + i < N) {
                    float *dst = dwr_partial + ((size_t)blockIdx.x * N + g0 + i) * d + c;
#pragma unroll
                    for (int u = 0; u < CPT; u += 4)
                        *reinterpret_cast<float4 *>(dst + u) = make_float4(acc[i][u], acc[i][u + 1], acc[i][u + 2], acc[i][u + 3]);
                }
        }
    }
}

// ---------------------------------------------------------------------------
// The same partial sums for bf16 layers on tensor cores (mma.sync m16n8k16): dW[e, c] = sum_t dz[t, e] x[t, c]
// is a [8 experts x 64 tokens] . [64 tokens x columns] product per token block.  dz is fp32: it enters as the
// sum of two bf16 numbers, hi = bf16(dz) in rows 0-7 of the A operand and lo = bf16(dz - hi) in rows 8-15, so one
// instruction forms both parts (x is bf16, every product is exact in fp32) and the two halves of the
// accumulator are added at the end; what is lost is below 2^-17 of each term.  A warp owns a unit of 64 tokens x
// 256 columns: it stages 32 columns at a time in shared memory (16-byte loads, rows padded to 80 bytes) and reads
// them back transposed with ldmatrix, which yields the B operand (pairs of consecutive tokens per column).  Units
// are dealt to the blocks round-robin, so every SM gets the same number of them (+-1).
// ---------------------------------------------------------------------------
constexpr int kDwrUnitCols = 256;
constexpr int kDwrChunkCols = 32;
constexpr int kDwrXPitch = 80;                       // bytes per staged row: 64 of data + 16 of skew (conflict-free ldmatrix)
constexpr int kDwrZPitch = 72;                       // bf16 per expert row of the dz slice: 64 tokens + 8 of skew
constexpr int kDwrWarpSmem = kDwrTokB * kDwrXPitch + 2 * 8 * kDwrZPitch * 2;   // x chunk + hi and lo slices of dz

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__global__ void __launch_bounds__(256)
router_dwr_mma_kernel(const __nv_bfloat16 *__restrict__ x, int Ttok, int d, int N, int k, const int *__restrict__ topk_idx,
                      const float *__restrict__ dz, float *__restrict__ dwr_partial, const float *__restrict__ logits,
                      const int *__restrict__ counts_slot, float aux_scale, const float *__restrict__ dense, int nblk,
                      int nslice)
{
    extern __shared__ __align__(16) unsigned char dwr_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, tq = lane & 3;
    unsigned char *xs = dwr_smem + (size_t)warp * kDwrWarpSmem;
    __nv_bfloat16 *zh = reinterpret_cast<__nv_bfloat16 *>(xs + kDwrTokB * kDwrXPitch);      // [8][kDwrZPitch]
    __nv_bfloat16 *zl = zh + 8 * kDwrZPitch;
    const uint32_t xs_addr = (uint32_t)__cvta_generic_to_shared(xs);
    const int units = nblk * nslice;
    const float inv_T = 1.0f / (float)Ttok;
    for (int u = blockIdx.x + gridDim.x * warp; u < units; u += gridDim.x * 8) {
        const int blk = u / nslice, slice = u - blk * nslice;
        const int t0 = blk * kDwrTokB;
        const int ntok = min(kDwrTokB, Ttok - t0);
        const int c_begin = slice * kDwrUnitCols, c_end = min(d, c_begin + kDwrUnitCols);
        for (int g0 = 0; g0 < N; g0 += 8) {
            // this group's slice of dz (dense over its 8 experts), split into hi and lo: a lane builds tokens lane, lane + 32
            __syncwarp();
            for (int tl = lane; tl < kDwrTokB; tl += 32) {
                float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (tl < ntok) {
                    const int t = t0 + tl;
                    if (dense != nullptr) {
                        for (int i = 0; i < 8; ++i)
                            if (g0 + i < N) v[i] = dense[(size_t)t * N + g0 + i];
                    } else {
                        for (int j = 0; j < k; ++j) {
                            const int e = topk_idx[(size_t)t * k + j] - g0;
                            const float dzv = dz[(size_t)t * k + j];
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if (e == i) v[i] = dzv;
                        }
                        if (aux_scale != 0.f) {
                            float zmax, inv_den, fp;
                            const float *zt = logits + (size_t)t * N;
                            token_softmax_stats(zt, counts_slot, N, inv_T, zmax, inv_den, fp);
                            for (int i = 0; i < 8; ++i)
                                if (g0 + i < N)
                                    v[i] += aux_scale * expf(zt[g0 + i] - zmax) * inv_den *
                                            ((float)counts_slot[g0 + i] * inv_T - fp);
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(v[i]);
                    zh[i * kDwrZPitch + tl] = hi;
                    zl[i * kDwrZPitch + tl] = __float2bfloat16_rn(v[i] - __bfloat162float(hi));
                }
            }
            __syncwarp();
            uint32_t af[4][4];                 // A fragments of the four 16-token steps
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                af[ks][0] = *reinterpret_cast<const uint32_t *>(zh + g * kDwrZPitch + 16 * ks + 2 * tq);
                af[ks][1] = *reinterpret_cast<const uint32_t *>(zl + g * kDwrZPitch + 16 * ks + 2 * tq);
                af[ks][2] = *reinterpret_cast<const uint32_t *>(zh + g * kDwrZPitch + 16 * ks + 2 * tq + 8);
                af[ks][3] = *reinterpret_cast<const uint32_t *>(zl + g * kDwrZPitch + 16 * ks + 2 * tq + 8);
            }
            // rows lane / 4 + 8 i of the staged chunk, 16-byte piece lane % 4
            auto fetch = [&](int c0, uint4 (&buf)[8]) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = (lane >> 2) + 8 * i;
                    buf[i] = (r < ntok && c0 < c_end)
                                 ? *reinterpret_cast<const uint4 *>(x + (size_t)(t0 + r) * d + c0 + (lane & 3) * 8)
                                 : make_uint4(0u, 0u, 0u, 0u);
                }
            };
            uint4 cur[8];
            fetch(c_begin, cur);
            for (int c0 = c_begin; c0 < c_end; c0 += kDwrChunkCols) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<uint4 *>(xs + ((lane >> 2) + 8 * i) * kDwrXPitch + (lane & 3) * 16) = cur[i];
                __syncwarp();
                fetch(c0 + kDwrChunkCols, cur);                   // the next chunk travels while this one is multiplied
                float acc[4][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                    for (int np = 0; np < 2; ++np) {
                        // matrix lane / 8: tokens 16 ks + 8 (m & 1) .., columns 16 np + 8 (m >> 1) ..
                        const int m = lane >> 3;
                        const uint32_t addr = xs_addr + (16 * ks + 8 * (m & 1) + (lane & 7)) * kDwrXPitch +
                                              (16 * np + 8 * (m >> 1)) * 2;
                        uint32_t b[4];
                        ldmatrix_x4_trans(b, addr);
                        mma_bf16_16816(acc[2 * np], af[ks][0], af[ks][1], af[ks][2], af[ks][3], b[0], b[1]);
                        mma_bf16_16816(acc[2 * np + 1], af[ks][0], af[ks][1], af[ks][2], af[ks][3], b[2], b[3]);
                    }
                }
                __syncwarp();                                     // the chunk has been read: it may be overwritten
                if (g0 + g < N) {
                    float *dst = dwr_partial + ((size_t)blk * N + g0 + g) * d + c0 + 2 * tq;
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt)
                        *reinterpret_cast<float2 *>(dst + nt * 8) =
                            make_float2(acc[nt][0] + acc[nt][2], acc[nt][1] + acc[nt][3]);
                }
            }
        }
    }
}

// Sums the per-block partials in a fixed order: warp p of a block adds the partials b = p, p + 8, ... of 32
// elements, then the eight warp sums are added in warp order.
__global__ void __launch_bounds__(256)
reduce_dwr_kernel(const float *__restrict__ partial, int nblk, int n, float *__restrict__ dwr)
{
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, p = threadIdx.x >> 5;
    const int i = blockIdx.x * 32 + lane;
    float s = 0.f;
    if (i < n) {
        // eight loads in flight at a time; the additions keep their order
        for (int b0 = p; b0 < nblk; b0 += 64) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = b0 + 8 * u < nblk ? partial[(size_t)(b0 + 8 * u) * n + i] : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (b0 + 8 * u < nblk) s += v[u];
        }
    }
    part[p][lane] = s;
    __syncthreads();
    if (p == 0 && i < n) {
        float acc = part[0][lane];
#pragma unroll
        for (int q = 1; q < 8; ++q) acc += part[q][lane];
        dwr[i] = acc;
    }
}

}  // namespace

// ---------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------
#define MODSE_LAUNCH_CHECK()                        \
    do {                                            \
        cudaError_t e__ = cudaGetLastError();       \
        if (e__ != cudaSuccess) return e__;         \
        if (launches) ++*launches;                  \
    } while (0)

cudaError_t launch_router(modse_dtype_t dt, const LayerMeta &m, const void *x, const void *w_router, int T,
                          const WsPtrs &p, const NoiseGate &ng, cudaStream_t s, int *launches)
{
    const int nblk = (T + kRouterTokB - 1) / kRouterTokB;
    const bool noise = ng.w_noise != nullptr;
    if (dt == MODSE_BF16 && m.N <= 16 && m.d % (32 * kRouterKSplit) == 0 && m.k * m.N * 4 <= 128) {
        const int nt = (m.N + 7) / 8, ntt = noise ? 2 * nt : nt;
        const size_t smem = 128 + (size_t)(kRouterKSplit - 1) * 4 * 32 * ntt * 4 * sizeof(float) +
                            (size_t)ntt * 8 * (m.d + 8) * 2;
        if (smem <= 200 * 1024 && !(noise && nt > 1)) {
            auto kern = noise ? router_mma_kernel<1, true>
                              : (nt == 1 ? router_mma_kernel<1, false> : router_mma_kernel<2, false>);
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            kern<<<nblk, kRouterMmaThreads, smem, s>>>((const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w_router, T, m.d, m.N, m.k,
                                         p.topk_idx, p.topk_gate, p.block_counts, p.logits,
                                         (const __nv_bfloat16 *)ng.w_noise, ng.gamma, ng.eps, p.noise_u, p.super_counts);
            MODSE_LAUNCH_CHECK();
            return cudaSuccess;
        }
    }
    const size_t esz = dt == MODSE_F32 ? 4 : 2;
    const size_t base = sizeof(int) * ((m.k * m.N + 3) & ~3) + sizeof(float) * 16 * ((m.N + 3) & ~3);
    const size_t wbytes = (size_t)m.N * m.d * esz * (noise ? 2 : 1);
    const int w_in_smem = (base + wbytes <= 160 * 1024) ? 1 : 0;
    const size_t smem = base + (w_in_smem ? wbytes : 0);
    if (dt == MODSE_F32) {
        auto kern = router_kernel<float>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<nblk, 256, smem, s>>>((const float *)x, (const float *)w_router, T, m.d, m.N, m.k, p.topk_idx,
                                     p.topk_gate, p.block_counts, p.logits, w_in_smem, (const float *)ng.w_noise,
                                     ng.gamma, ng.eps, p.noise_u, p.super_counts);
    } else {
        auto kern = router_kernel<__nv_bfloat16>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<nblk, 256, smem, s>>>((const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w_router, T, m.d, m.N, m.k,
                                     p.topk_idx, p.topk_gate, p.block_counts, p.logits, w_in_smem,
                                     (const __nv_bfloat16 *)ng.w_noise, ng.gamma, ng.eps, p.noise_u, p.super_counts);
    }
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

cudaError_t launch_rank(const LayerMeta &m, int T, int Pmax, const WsPtrs &p, cudaStream_t s, int *launches)
{
    const int nblk = (T + kRouterTokB - 1) / kRouterTokB;
    const int kN = m.k * m.N;
    const size_t smem = sizeof(int) * (2 * kN + 2 * (m.N + 1) + m.N + kRouterTokB * m.k);
    rank_kernel<<<nblk, 256, smem, s>>>(m, T, Pmax, nblk, p.block_counts, p.super_counts, p.topk_idx, p.topk_gate, p.counts,
                                        p.counts_slot, p.offsets, p.poffsets, p.ebase, p.row_of, p.token_of,
                                        p.prow_of, p.ptoken_of, p.pgate, p.status);
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

cudaError_t launch_permute(modse_dtype_t dt, const LayerMeta &m, const void *x, int T, int Pmax, const WsPtrs &p,
                           cudaStream_t s, int *launches)
{
    const int tok_blocks = (T + 7) / 8;
    const int grid = tok_blocks + m.N * 16;
    if (dt == MODSE_F32)
        permute_kernel<float><<<grid, 256, 0, s>>>((const float *)x, T, m.d, m.N, m.k, p.prow_of, p.counts,
                                                   p.poffsets, (float *)p.xp, tok_blocks, Pmax, p.status);
    else
        permute_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)x, T, m.d, m.N, m.k, p.prow_of,
                                                           p.counts, p.poffsets, (__nv_bfloat16 *)p.xp, tok_blocks,
                                                           Pmax, p.status);
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

cudaError_t launch_combine(modse_dtype_t dt, const LayerMeta &m, int T, int Pmax, const WsPtrs &p, void *y, bool out_f32,
                           cudaStream_t s, int *launches)
{
    const int grid = (T + 7) / 8;
    if (dt == MODSE_F32 || out_f32)
        combine_kernel<float><<<grid, 256, 0, s>>>((const float *)p.o, T, m.d, m.k, p.prow_of, (float *)y, Pmax,
                                                   p.status);
    else
        combine_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const float *)p.o, T, m.d, m.k, p.prow_of,
                                                           (__nv_bfloat16 *)y, Pmax, p.status);
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

template <typename T, bool WITH_DG>
static void launch_dg_permute_t(const LayerMeta &m, const void *dy, int Ttok, int Pmax, const WsPtrs &p, cudaStream_t s)
{
    const int tok_blocks = (Ttok + 7) / 8;
    const int grid = tok_blocks + m.N * 16;
    dg_permute_kernel<T, WITH_DG><<<grid, 256, 0, s>>>((const T *)dy, (const float *)p.o, Ttok, m.d, m.N, m.k, p.prow_of,
                                                       p.topk_gate, p.counts, p.poffsets, p.dg, (T *)p.dyp, tok_blocks,
                                                       Pmax, p.status);
}

cudaError_t launch_dg_permute(modse_dtype_t dt, const LayerMeta &m, const void *dy, int T, int Pmax, const WsPtrs &p,
                              bool with_dg, cudaStream_t s, int *launches)
{
    if (dt == MODSE_F32) {
        if (with_dg) launch_dg_permute_t<float, true>(m, dy, T, Pmax, p, s);
        else launch_dg_permute_t<float, false>(m, dy, T, Pmax, p, s);
    } else {
        if (with_dg) launch_dg_permute_t<__nv_bfloat16, true>(m, dy, T, Pmax, p, s);
        else launch_dg_permute_t<__nv_bfloat16, false>(m, dy, T, Pmax, p, s);
    }
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

// Guard blocks between the workspace regions: block i holds kCanaryPattern ^ i in its first 8 bytes.
struct CanaryOffsets {
    int n;
    size_t off[kMaxCanaries];
};
namespace {
__global__ void canary_kernel(unsigned char *ws, CanaryOffsets c, int check, int *status)
{
    const int i = threadIdx.x;
    if (i >= c.n) return;
    unsigned long long *w = reinterpret_cast<unsigned long long *>(ws + c.off[i]);
    const unsigned long long want = kCanaryPattern ^ (unsigned long long)i;
    if (!check) *w = want;
    else if (*w != want) atomicMax(status, kDevBounds);
}
}  // namespace

cudaError_t launch_canaries(void *ws, const WsLayout &L, bool check, int *status, cudaStream_t s)
{
    CanaryOffsets c;
    c.n = L.n_canary;
    for (int i = 0; i < kMaxCanaries; ++i) c.off[i] = i < L.n_canary ? L.canary[i] : 0;
    canary_kernel<<<1, 64, 0, s>>>(static_cast<unsigned char *>(ws), c, check ? 1 : 0, status);
    return cudaGetLastError();
}

cudaError_t launch_router_bwd(modse_dtype_t dt, const LayerMeta &m, const void *x, const void *w_router, int T,
                              int Pmax, int nblk_bwd, const WsPtrs &p, void *dx, bool out_f32, bool dx_holds_sum,
                              float *dw_router, float aux_scale, const NoiseGate &ng, cudaStream_t s, int *launches)
{
    const int hs = dx_holds_sum ? 1 : 0;
    const bool noise = ng.w_noise != nullptr;
    const float *du = noise ? p.du : nullptr;
    if (noise) {
        noise_bwd_kernel<<<nblk_bwd, kRouterBwdTokB, 0, s>>>(p.noise_u, T, m.N, m.k, p.topk_idx, p.topk_gate, p.dg,
                                                             p.logits, p.counts_slot, aux_scale, ng.gamma, ng.eps,
                                                             p.du, p.dgamma_partial);
        MODSE_LAUNCH_CHECK();
        reduce_scalar_kernel<<<1, 32, 0, s>>>(p.dgamma_partial, nblk_bwd, ng.dgamma);
        MODSE_LAUNCH_CHECK();
    }
    const int grid_dx = (T + 7) / 8;
    const float *dxp = (const float *)p.dxp;
    if (dt == MODSE_F32)
        router_dx_kernel<float, float><<<grid_dx, 256, 0, s>>>((const float *)w_router, dxp, T, m.d, m.k, p.topk_idx,
                                                               p.topk_gate, p.prow_of, p.dg, p.dz, (float *)dx, m.N, p.logits,
                                                               p.counts_slot, aux_scale, (const float *)ng.w_noise, du,
                                                               Pmax, hs, p.status);
    else if (out_f32)
        router_dx_kernel<__nv_bfloat16, float><<<grid_dx, 256, 0, s>>>((const __nv_bfloat16 *)w_router, dxp, T, m.d,
                                                                       m.k, p.topk_idx, p.topk_gate, p.prow_of, p.dg,
                                                                       p.dz, (float *)dx, m.N, p.logits, p.counts_slot,
                                                                       aux_scale, (const __nv_bfloat16 *)ng.w_noise, du,
                                                                       Pmax, hs, p.status);
    else
        router_dx_kernel<__nv_bfloat16, __nv_bfloat16><<<grid_dx, 256, 0, s>>>(
            (const __nv_bfloat16 *)w_router, dxp, T, m.d, m.k, p.topk_idx, p.topk_gate, p.prow_of, p.dg, p.dz,
            (__nv_bfloat16 *)dx, m.N, p.logits, p.counts_slot, aux_scale, (const __nv_bfloat16 *)ng.w_noise, du, Pmax, hs,
            p.status);
    MODSE_LAUNCH_CHECK();
    const int nblk_dwr = (T + kDwrTokB - 1) / kDwrTokB;
    dim3 grid(nblk_dwr, dt == MODSE_F32 ? (m.d + 1023) / 1024 : (m.d + 2047) / 2048);
    const int n = m.N * m.d;
    // pass 0: dW_router = dz^T x;  pass 1 (second term only): dW_n = du^T x through the same partial buffer
    for (int pass = 0; pass < (noise ? 2 : 1); ++pass) {
        const float *dense = pass ? du : nullptr;
        const float ascale = pass ? 0.f : aux_scale;
        if (dt == MODSE_F32) {
            router_dwr_kernel<float><<<grid, 256, 0, s>>>((const float *)x, T, m.d, m.N, m.k, p.topk_idx, p.dz,
                                                          p.dwr_partial, p.logits, p.counts_slot, ascale, dense);
        } else if (m.d % kDwrChunkCols == 0) {
            // tensor-core form: units of 64 tokens x 256 columns, one per warp, dealt round-robin to the blocks
            const int nslice = (m.d + kDwrUnitCols - 1) / kDwrUnitCols;
            const int units = nblk_dwr * nslice;
            int dev = 0, sms = 0;
            if (cudaGetDevice(&dev) != cudaSuccess ||
                cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
                sms = 148;
            const int grid_mma = std::max(1, std::min(units, 2 * sms));     // two blocks of 118 registers x 256 threads per SM
            const size_t smem = (size_t)8 * kDwrWarpSmem;
            static bool attr_done = false;
            if (!attr_done) {
                cudaError_t e = cudaFuncSetAttribute(router_dwr_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)smem);
                if (e != cudaSuccess) return e;
                attr_done = true;
            }
            router_dwr_mma_kernel<<<grid_mma, 256, smem, s>>>((const __nv_bfloat16 *)x, T, m.d, m.N, m.k, p.topk_idx, p.dz,
                                                             p.dwr_partial, p.logits, p.counts_slot, ascale, dense,
                                                             nblk_dwr, nslice);
        } else {
            router_dwr_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)x, T, m.d, m.N, m.k,
                                                                  p.topk_idx, p.dz, p.dwr_partial, p.logits,
                                                                  p.counts_slot, ascale, dense);
        }
        MODSE_LAUNCH_CHECK();
        reduce_dwr_kernel<<<(n + 31) / 32, 256, 0, s>>>(p.dwr_partial, nblk_dwr, n, pass ? ng.dw_noise : dw_router);
        MODSE_LAUNCH_CHECK();
    }
    return cudaSuccess;
}

cudaError_t launch_aux_loss(const LayerMeta &m, int T, int nblk_bwd, const WsPtrs &p, float alpha, float *loss,
                            float *f, float *P, cudaStream_t s, int *launches)
{
    aux_partial_kernel<<<nblk_bwd, 128, 0, s>>>(p.logits, T, m.N, p.aux_partial);
    MODSE_LAUNCH_CHECK();
    aux_final_kernel<<<1, 256, 0, s>>>(p.aux_partial, nblk_bwd, p.counts_slot, T, m.N, alpha, loss, f, P);
    MODSE_LAUNCH_CHECK();
    return cudaSuccess;
}

}  // namespace modse
