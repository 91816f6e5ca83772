// fp32-FMA grouped GEMMs over the padded expert groups, and the SwiGLU
// elementwise stages.  This is the arithmetic path of the fp32 layer type
// (fp32 storage needs full-precision products, which the bf16 tensor-core
// pipeline cannot give); with bf16 storage it doubles as a slow cross-check of
// the tensor-core kernels.
//
// Every product is C_e(m,n) (+)= sum_k A_e(m,k) * B_e(n,k), k ascending, one
// problem per expert, operands addressed through (row, column) strides so that
// the transposed uses in the backward pass need no copies.
#include "modse_internal.h"

namespace modse {

namespace {

struct Problem {
    const void *A, *B;
    void *C;
    long long a_rs, a_cs, b_rs, b_cs, c_rs;
    int M, Nn, K;
};

__device__ __forceinline__ float ld(const float *p, long long i) { return p[i]; }
__device__ __forceinline__ float ld(const __nv_bfloat16 *p, long long i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st(float *p, long long i, float v) { p[i] = v; }
__device__ __forceinline__ void st(__nv_bfloat16 *p, long long i, float v) { p[i] = __float2bfloat16_rn(v); }

// Results that are later summed over a token's slots (o of kDown, dxp of
// kUpGateDgrad) are fp32 buffers whatever the layer type.
__host__ __device__ inline bool out_is_f32(int kind) { return kind == kDown || kind == kUpGateDgrad; }

template <typename T>
__device__ Problem make_problem(int kind, const LayerMeta &m, int e, const int *poffsets, const long long *ebase,
                                const T *act, const T *wgt, void *out_v)
{
    const long long d = m.d, S = m.S;
    const long long ho = m.hoff[e], he = m.hoff[e + 1] - m.hoff[e];
    const long long po = poffsets[e], cp = poffsets[e + 1] - poffsets[e];
    const long long eb = ebase[e];
    T *out = static_cast<T *>(out_v);
    float *outf = static_cast<float *>(out_v);
    Problem p;
    switch (kind) {
    case kUpGate:       // C[cp,he] = xp . W^T
        p.A = act + po * d; p.a_rs = d; p.a_cs = 1;
        p.B = wgt + ho * d; p.b_rs = d; p.b_cs = 1;
        p.C = out + eb; p.c_rs = he; p.M = (int)cp; p.Nn = (int)he; p.K = (int)d;
        break;
    case kDown:         // o[cp,d] = Hm . W_down_e^T, W_down is [d,S]
        p.A = act + eb; p.a_rs = he; p.a_cs = 1;
        p.B = wgt + ho; p.b_rs = S; p.b_cs = 1;
        p.C = outf + po * d; p.c_rs = d; p.M = (int)cp; p.Nn = (int)d; p.K = (int)he;
        break;
    case kDownDgrad:    // dHm[cp,he] = dyp . W_down_e ; B(n,k) = W_down[k, ho+n]
        p.A = act + po * d; p.a_rs = d; p.a_cs = 1;
        p.B = wgt + ho; p.b_rs = 1; p.b_cs = S;
        p.C = out + eb; p.c_rs = he; p.M = (int)cp; p.Nn = (int)he; p.K = (int)d;
        break;
    case kDownWgrad:    // dW_down[q, ho+r] = sum_i dyp[i,q] Hm[i,r]
        p.A = act + po * d; p.a_rs = 1; p.a_cs = d;
        p.B = wgt + eb; p.b_rs = 1; p.b_cs = he;
        p.C = out + ho; p.c_rs = S; p.M = (int)d; p.Nn = (int)he; p.K = (int)cp;
        break;
    case kUpGateDgrad:  // dxp[cp,d] (+)= dA . W ; B(n,k) = W[ho+k, n]
        p.A = act + eb; p.a_rs = he; p.a_cs = 1;
        p.B = wgt + ho * d; p.b_rs = 1; p.b_cs = d;
        p.C = outf + po * d; p.c_rs = d; p.M = (int)cp; p.Nn = (int)d; p.K = (int)he;
        break;
    default:            // kUpGateWgrad: dW[ho+r, c] = sum_i dA[i,r] xp[i,c]
        p.A = act + eb; p.a_rs = 1; p.a_cs = he;
        p.B = wgt + po * d; p.b_rs = 1; p.b_cs = d;
        p.C = out + ho * d; p.c_rs = d; p.M = (int)he; p.Nn = (int)d; p.K = (int)cp;
        break;
    }
    return p;
}

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__global__ void __launch_bounds__(256)
simt_grouped_gemm(int kind, LayerMeta m, const int *__restrict__ poffsets, const long long *__restrict__ ebase,
                  const T *act, const T *wgt, void *out, int accumulate)
{
    const int e = blockIdx.z;
    const Problem p = make_problem<T>(kind, m, e, poffsets, ebase, act, wgt, out);
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (m0 >= p.M || n0 >= p.Nn) return;
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN + 1];
    const T *A = static_cast<const T *>(p.A);
    const T *B = static_cast<const T *>(p.B);
    T *C = static_cast<T *>(p.C);
    float *Cf = static_cast<float *>(p.C);
    const bool f32out = out_is_f32(kind);
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4] = {};
    // Loader mapping: the fast thread index follows the operand's contiguous axis.
    const bool a_kfast = (p.a_cs == 1), b_kfast = (p.b_cs == 1);
    for (int k0 = 0; k0 < p.K; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int l = tid + i * 256;
            const int kk = a_kfast ? (l % BK) : (l / BM);
            const int mm = a_kfast ? (l / BK) : (l % BM);
            float v = 0.f;
            if (m0 + mm < p.M && k0 + kk < p.K) v = ld(A, (long long)(m0 + mm) * p.a_rs + (long long)(k0 + kk) * p.a_cs);
            As[kk][mm] = v;
            const int kb = b_kfast ? (l % BK) : (l / BN);
            const int nn = b_kfast ? (l / BK) : (l % BN);
            v = 0.f;
            if (n0 + nn < p.Nn && k0 + kb < p.K) v = ld(B, (long long)(n0 + nn) * p.b_rs + (long long)(k0 + kb) * p.b_cs);
            Bs[kb][nn] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int mm = m0 + ty * 4 + i;
        if (mm >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int nn = n0 + tx * 4 + j;
            if (nn >= p.Nn) continue;
            const long long idx = (long long)mm * p.c_rs + nn;
            float v = acc[i][j];
            if (f32out) {
                if (accumulate) v += Cf[idx];
                Cf[idx] = v;
            } else {
                if (accumulate) v += ld(C, idx);
                st(C, idx, v);
            }
        }
    }
}

// hm[r,:] = g_r * silu(a[r,:]) * b[r,:] for every padded row r of every expert
// (g_r = gate of the assignment in that row, 0 for padding rows).
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_fwd_kernel(const T *__restrict__ a, const T *__restrict__ b, T *__restrict__ hm, LayerMeta m,
                  const int *__restrict__ poffsets, const long long *__restrict__ ebase,
                  const float *__restrict__ pgate)
{
    const int e = blockIdx.y;
    const int he = m.hoff[e + 1] - m.hoff[e];
    const int cp = poffsets[e + 1] - poffsets[e];
    const long long n = (long long)cp * he, eb = ebase[e];
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const float g = pgate[poffsets[e] + (int)(i / he)];
        const float av = ld(a, eb + i), bv = ld(b, eb + i);
        const float sg = 1.0f / (1.0f + expf(-av));
        st(hm, eb + i, g * (av * sg * bv));
    }
}

// dhm = g_r * (dY W_down) arrives ungated in the da buffer;
// da = dhm * b * silu'(a), db = dhm * silu(a).
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_bwd_kernel(const T *__restrict__ a, const T *__restrict__ b, T *__restrict__ da, T *__restrict__ db,
                  LayerMeta m, const int *__restrict__ poffsets, const long long *__restrict__ ebase,
                  const float *__restrict__ pgate)
{
    const int e = blockIdx.y;
    const int he = m.hoff[e + 1] - m.hoff[e];
    const int cp = poffsets[e + 1] - poffsets[e];
    const long long n = (long long)cp * he, eb = ebase[e];
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const float g = pgate[poffsets[e] + (int)(i / he)];
        const float av = ld(a, eb + i), bv = ld(b, eb + i), dh = g * ld(da, eb + i);
        const float sg = 1.0f / (1.0f + expf(-av));
        st(da, eb + i, dh * bv * sg * (1.0f + av * (1.0f - sg)));
        st(db, eb + i, dh * av * sg);
    }
}

}  // namespace

cudaError_t launch_simt_gemm(modse_dtype_t dt, GemmKind kind, const LayerMeta &m, int Pmax, const WsPtrs &p,
                             const SimtGemmArgs &a, cudaStream_t s, int *launches)
{
    int hmax = 0;
    for (int e = 0; e < m.N; ++e) hmax = max(hmax, m.hoff[e + 1] - m.hoff[e]);
    int Mmax, Nmax;
    switch (kind) {
    case kUpGate: case kDownDgrad: Mmax = Pmax; Nmax = hmax; break;
    case kDown: case kUpGateDgrad: Mmax = Pmax; Nmax = m.d; break;
    case kDownWgrad: Mmax = m.d; Nmax = hmax; break;
    default: Mmax = hmax; Nmax = m.d; break;
    }
    dim3 grid((Nmax + BN - 1) / BN, (Mmax + BM - 1) / BM, m.N);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    if (dt == MODSE_F32)
        simt_grouped_gemm<float><<<grid, 256, 0, s>>>((int)kind, m, p.poffsets, p.ebase, (const float *)a.act,
                                                      (const float *)a.wgt, a.out, a.accumulate);
    else
        simt_grouped_gemm<__nv_bfloat16><<<grid, 256, 0, s>>>((int)kind, m, p.poffsets, p.ebase,
                                                              (const __nv_bfloat16 *)a.act,
                                                              (const __nv_bfloat16 *)a.wgt, a.out, a.accumulate);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (launches) ++*launches;
    return cudaSuccess;
}

cudaError_t launch_swiglu_fwd(modse_dtype_t dt, const LayerMeta &m, const WsPtrs &p, size_t hb, cudaStream_t s,
                              int *launches)
{
    (void)hb;
    dim3 grid(148, m.N);
    if (dt == MODSE_F32)
        swiglu_fwd_kernel<float><<<grid, 256, 0, s>>>((const float *)p.a_pre, (const float *)p.b_pre, (float *)p.hm, m,
                                                      p.poffsets, p.ebase, p.pgate);
    else
        swiglu_fwd_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)p.a_pre,
                                                              (const __nv_bfloat16 *)p.b_pre,
                                                              (__nv_bfloat16 *)p.hm, m, p.poffsets, p.ebase, p.pgate);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (launches) ++*launches;
    return cudaSuccess;
}

cudaError_t launch_swiglu_bwd(modse_dtype_t dt, const LayerMeta &m, const WsPtrs &p, size_t hb, cudaStream_t s,
                              int *launches)
{
    (void)hb;
    dim3 grid(148, m.N);
    if (dt == MODSE_F32)
        swiglu_bwd_kernel<float><<<grid, 256, 0, s>>>((const float *)p.a_pre, (const float *)p.b_pre, (float *)p.da,
                                                      (float *)p.db, m, p.poffsets, p.ebase, p.pgate);
    else
        swiglu_bwd_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)p.a_pre,
                                                              (const __nv_bfloat16 *)p.b_pre,
                                                              (__nv_bfloat16 *)p.da, (__nv_bfloat16 *)p.db, m,
                                                              p.poffsets, p.ebase, p.pgate);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (launches) ++*launches;
    return cudaSuccess;
}

}  // namespace modse
