// Winograd transform kernels (Eq. 6): U = G w G^T, V = B^T d B, y = act(A^T M A + bias).
// The matrices come from the host generator (Eq. 8) as kernel parameters, so any
// point set works; the kernels are instantiated per alpha (and m for the output
// side) so that a tile lives in registers.
#include <cuda_bf16.h>

#include "kernels.h"
#include "wino_transforms.cuh"

MNNB_DECLARE_INPUT(3) MNNB_DECLARE_INPUT(4) MNNB_DECLARE_INPUT(5) MNNB_DECLARE_INPUT(6)
MNNB_DECLARE_INPUT(7) MNNB_DECLARE_INPUT(8) MNNB_DECLARE_INPUT(10) MNNB_DECLARE_INPUT(12)
MNNB_DECLARE_OUTPUT(3, 2) MNNB_DECLARE_OUTPUT(5, 4) MNNB_DECLARE_OUTPUT(7, 6)
MNNB_DECLARE_OUTPUT(4, 2) MNNB_DECLARE_OUTPUT(6, 4) MNNB_DECLARE_OUTPUT(8, 6)
MNNB_DECLARE_OUTPUT(6, 2) MNNB_DECLARE_OUTPUT(8, 4) MNNB_DECLARE_OUTPUT(10, 6)
MNNB_DECLARE_OUTPUT(8, 2) MNNB_DECLARE_OUTPUT(10, 4) MNNB_DECLARE_OUTPUT(12, 6)

namespace mnnb {

using wino::MatG;
using wino::store_operand;

namespace {

// ---------------------------------------------------------------------------
// Weight transform: one thread per (co, ci); preparation time only.
// ---------------------------------------------------------------------------
__global__ void weight_transform_kernel(const float* __restrict__ w, void* U_hi, void* U_lo, int Cout, int Cin, int k,
                                        int alpha, int cin_pad, int mode, MatG G)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)Cout * cin_pad;
    if (gid >= total) return;
    const int ci = (int)(gid % cin_pad), co = (int)(gid / cin_pad);
    float g[49];
    float t[12 * 7];
    const bool real = ci < Cin;
    for (int e = 0; e < k * k; ++e) g[e] = real ? w[((size_t)co * Cin + ci) * k * k + e] : 0.0f;
    for (int i = 0; i < alpha; ++i)
        for (int b = 0; b < k; ++b) {
            float s = 0.0f;
            for (int a = 0; a < k; ++a) s = fmaf(G.v[i * k + a], g[a * k + b], s);
            t[i * k + b] = s;
        }
    for (int i = 0; i < alpha; ++i)
        for (int j = 0; j < alpha; ++j) {
            float s = 0.0f;
            for (int b = 0; b < k; ++b) s = fmaf(t[i * k + b], G.v[j * k + b], s);
            const size_t idx = ((size_t)(i * alpha + j) * Cout + co) * cin_pad + ci;
            store_operand(U_hi, U_lo, idx, s, mode);
        }
}

__global__ void weight_round_kernel(const float* __restrict__ w, void* U_hi, void* U_lo, int Cout, int Kd, int k_pad,
                                    int mode)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)Cout * k_pad;
    if (gid >= total) return;
    const int kk = (int)(gid % k_pad), co = (int)(gid / k_pad);
    const float v = kk < Kd ? w[(size_t)co * Kd + kk] : 0.0f;
    store_operand(U_hi, U_lo, (size_t)gid, v, mode);
}

// ---------------------------------------------------------------------------
// CUDA-core fp32 contraction (checking path): one thread per (t, co, xi).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float load_operand(const void* hi, const void* lo, size_t idx, int mode)
{
    switch (mode) {
        case STORE_BF16:
            return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(hi)[idx]);
        case STORE_TF32_SPLIT:
            return reinterpret_cast<const float*>(hi)[idx] + reinterpret_cast<const float*>(lo)[idx];
        case STORE_BF16_SPLIT:
            return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(hi)[idx]) +
                   __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(lo)[idx]);
        default:
            return reinterpret_cast<const float*>(hi)[idx];
    }
}

__global__ void contract_reference_kernel(const void* U_hi, const void* U_lo, const void* V_hi, const void* V_lo, int mode,
                                          int Cout, long long tiles, int cin_pad, long long u_plane, long long v_plane,
                                          ContractEpilogue epi)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int co = blockIdx.y, xi = blockIdx.z;
    if (t >= tiles) return;
    float s = 0.0f;
    const size_t ub = (size_t)xi * u_plane + (size_t)co * cin_pad;
    const size_t vb = (size_t)xi * v_plane + (size_t)t * cin_pad;
    for (int c = 0; c < cin_pad; ++c)
        s = fmaf(load_operand(U_hi, U_lo, ub + c, mode), load_operand(V_hi, V_lo, vb + c, mode), s);
    if (epi.mode == 0) {
        epi.M[((size_t)xi * Cout + co) * epi.m_row_stride + t] = s;
    } else {
        const long long n = t / epi.ohw, pix = t % epi.ohw;
        s += epi.bias ? epi.bias[co] : 0.0f;
        if (epi.relu) s = fmaxf(s, 0.0f);
        epi.y[((size_t)n * Cout + co) * epi.ohw + pix] = s;
    }
}

}  // namespace

cudaError_t launch_weight_transform(const float* w, void* U_hi, void* U_lo, int Cout, int Cin, int k, int m, int cin_pad,
                                    int mode, const TransformMatrices& mats, cudaStream_t stream)
{
    const int alpha = m + k - 1;
    if (alpha > 12 || k > 7) return cudaErrorInvalidValue;
    MatG G;
    for (int i = 0; i < alpha * k; ++i) G.v[i] = mats.G[i];
    const long long total = (long long)Cout * cin_pad;
    const int threads = 128;
    weight_transform_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, stream>>>(w, U_hi, U_lo, Cout, Cin, k,
                                                                                                 alpha, cin_pad, mode, G);
    return cudaGetLastError();
}

cudaError_t launch_weight_round(const float* w, void* U_hi, void* U_lo, int Cout, int Kd, int k_pad, int mode,
                                cudaStream_t stream)
{
    const long long total = (long long)Cout * k_pad;
    const int threads = 256;
    weight_round_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, stream>>>(w, U_hi, U_lo, Cout, Kd, k_pad,
                                                                                             mode);
    return cudaGetLastError();
}

cudaError_t launch_input_transform(const float* x, void* V_hi, void* V_lo, const WinoGeom& g, int mode,
                                   const TransformMatrices& mats, int* status, cudaStream_t stream)
{
    static int num_sms = 0;
    if (num_sms == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            n <= 0)
            n = 148;
        num_sms = n;
    }
    switch (g.alpha) {
        case 3: return MNNB_INPUT_FN(3)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 4: return MNNB_INPUT_FN(4)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 5: return MNNB_INPUT_FN(5)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 6: return MNNB_INPUT_FN(6)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 7: return MNNB_INPUT_FN(7)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 8: return MNNB_INPUT_FN(8)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 10: return MNNB_INPUT_FN(10)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        case 12: return MNNB_INPUT_FN(12)(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_output_transform(const float* M, const float* bias, float* y, const WinoGeom& g, int relu,
                                    const TransformMatrices& mats, cudaStream_t stream)
{
#define MNNB_OUT_CASE(A, MM) \
    if (g.alpha == A && g.m == MM) return MNNB_OUTPUT_FN(A, MM)(M, bias, y, g, relu, mats, stream);
    MNNB_OUT_CASE(3, 2) MNNB_OUT_CASE(5, 4) MNNB_OUT_CASE(7, 6)       // k = 2
    MNNB_OUT_CASE(4, 2) MNNB_OUT_CASE(6, 4) MNNB_OUT_CASE(8, 6)       // k = 3
    MNNB_OUT_CASE(6, 2) MNNB_OUT_CASE(8, 4) MNNB_OUT_CASE(10, 6)      // k = 5
    MNNB_OUT_CASE(8, 2) MNNB_OUT_CASE(10, 4) MNNB_OUT_CASE(12, 6)     // k = 7
#undef MNNB_OUT_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_contract_reference(const void* U_hi, const void* U_lo, const void* V_hi, const void* V_lo, int mode,
                                      int alpha2, int Cout, long long tiles, int cin_pad, long long u_plane,
                                      long long v_plane, const ContractEpilogue& epi, cudaStream_t stream)
{
    if (tiles <= 0) return cudaSuccess;
    if (Cout > 65535 || alpha2 > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((tiles + 127) / 128), (unsigned)Cout, (unsigned)alpha2);
    contract_reference_kernel<<<grid, 128, 0, stream>>>(U_hi, U_lo, V_hi, V_lo, mode, Cout, tiles, cin_pad, u_plane, v_plane,
                                                        epi);
    return cudaGetLastError();
}

}  // namespace mnnb
