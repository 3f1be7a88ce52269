// One level of Strassen's algorithm around the tensor-core contraction (Section 3.3.2).
//
// C = A B with A = w [Cout x Cin], B = x [Cin x T] (T = N * H * W, a 1x1 convolution).  With the quadrants
// A_ij (i: half of Cout, j: half of Cin) and B_jk (k: half of the batch) the seven products are
//   M1 = (A11 + A22)(B11 + B22)   M2 = (A21 + A22) B11      M3 = A11 (B12 - B22)    M4 = A22 (B21 - B11)
//   M5 = (A11 + A12) B22          M6 = (A21 - A11)(B11 + B12)   M7 = (A12 - A22)(B21 + B22)
// and  C11 = M1 + M4 - M5 + M7,  C12 = M3 + M5,  C21 = M2 + M4,  C22 = M1 - M2 + M3 + M6.
// This is a bilinear algorithm of the same shape as Eq. 6: a transform of each operand (here: additions of
// quadrants), seven independent matrix products (run as ONE launch of the batched contraction, with seven
// "transform positions"), and a transform of the products.  The additions are therefore folded into one pass
// over x before and one pass over the products after the contraction; their number (the paper counts 15 for
// its variant, this form has 18) does not change the memory traffic of those passes.
#include "strassen.h"

#include <cuda_bf16.h>

#include "wino_transforms.cuh"

namespace mnnb {

namespace {

using wino::store_operand;

__global__ void strassen_weights_kernel(const float* __restrict__ w, void* U_hi, void* U_lo, int Cin, int Mh, int Kh, int k_pad,
                                        int mode)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)Mh * k_pad) return;
    const int c = (int)(gid % k_pad), co = (int)(gid / k_pad);
    float a11 = 0.f, a12 = 0.f, a21 = 0.f, a22 = 0.f;
    if (c < Kh) {
        a11 = w[(size_t)co * Cin + c];
        a12 = w[(size_t)co * Cin + Kh + c];
        a21 = w[(size_t)(Mh + co) * Cin + c];
        a22 = w[(size_t)(Mh + co) * Cin + Kh + c];
    }
    const float u[7] = {a11 + a22, a21 + a22, a11, a22, a11 + a12, a21 - a11, a12 - a22};
    const size_t plane = (size_t)Mh * k_pad;
#pragma unroll
    for (int xi = 0; xi < 7; ++xi) store_operand(U_hi, U_lo, xi * plane + (size_t)gid, u[xi], mode);
}

// One CTA: 32 pixels x 32 channels of the four quadrants, transposed through shared memory so that both the
// reads of x (pixel-contiguous) and the writes of V (channel-contiguous) are coalesced.
__global__ void __launch_bounds__(256) strassen_input_kernel(const float* __restrict__ x, void* V_hi, void* V_lo, StrassenGeom g,
                                                             int Kh, int mode)
{
    __shared__ float s[4][32][33];
    const int p0 = blockIdx.x * 32, c0 = blockIdx.y * 32, n = blockIdx.z;       // n: image of the first batch half
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;                      // 8 rows of threads
    const int Nh = g.N / 2;
    for (int q = 0; q < 4; ++q) {
        const int j = q >> 1, k = q & 1;                                         // quadrant B_jk
        const float* src = x + ((size_t)(k * Nh + n) * g.Cin + (size_t)j * Kh) * g.HW;
        for (int r = ty; r < 32; r += 8) {
            const int c = c0 + r, p = p0 + tx;
            s[q][r][tx] = (c < Kh && p < g.HW) ? __ldg(src + (size_t)c * g.HW + p) : 0.0f;
        }
    }
    __syncthreads();
    const size_t plane = (size_t)g.t_half * g.k_pad;
    for (int r = ty; r < 32; r += 8) {
        const int p = p0 + r, c = c0 + tx;
        if (p >= g.HW || c >= g.k_pad) continue;
        const float b11 = s[0][tx][r], b12 = s[1][tx][r], b21 = s[2][tx][r], b22 = s[3][tx][r];
        const float v[7] = {b11 + b22, b11, b12 - b22, b21 - b11, b22, b11 + b12, b21 + b22};
        const size_t idx = ((size_t)n * g.HW + p) * g.k_pad + c;
#pragma unroll
        for (int xi = 0; xi < 7; ++xi) store_operand(V_hi, V_lo, xi * plane + idx, v[xi], mode);
    }
}

__global__ void strassen_output_kernel(const float* __restrict__ M, const float* __restrict__ bias, float* __restrict__ y,
                                       StrassenGeom g, int Mh, int relu)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int co = blockIdx.y;
    if (t >= g.t_half) return;
    const size_t plane = (size_t)Mh * g.m_row_stride;
    const float* src = M + (size_t)co * g.m_row_stride + t;
    float m[7];
#pragma unroll
    for (int xi = 0; xi < 7; ++xi) m[xi] = __ldcs(src + xi * plane);
    const float c11 = m[0] + m[3] - m[4] + m[6], c12 = m[2] + m[4], c21 = m[1] + m[3], c22 = m[0] - m[1] + m[2] + m[5];
    const int Nh = g.N / 2;
    const long long n = t / g.HW, p = t - n * g.HW;
    const float b0 = bias ? __ldg(bias + co) : 0.0f, b1 = bias ? __ldg(bias + Mh + co) : 0.0f;
    float o[4] = {c11 + b0, c12 + b0, c21 + b1, c22 + b1};
    if (relu) {
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = fmaxf(o[i], 0.0f);
    }
    y[((size_t)n * g.Cout + co) * g.HW + p] = o[0];
    y[((size_t)(Nh + n) * g.Cout + co) * g.HW + p] = o[1];
    y[((size_t)n * g.Cout + Mh + co) * g.HW + p] = o[2];
    y[((size_t)(Nh + n) * g.Cout + Mh + co) * g.HW + p] = o[3];
}

}  // namespace

cudaError_t launch_strassen_weights(const float* w, void* U_hi, void* U_lo, const StrassenGeom& g, int mode, cudaStream_t stream)
{
    const int Mh = g.Cout / 2, Kh = g.Cin / 2;
    const long long total = (long long)Mh * g.k_pad;
    strassen_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(w, U_hi, U_lo, g.Cin, Mh, Kh, g.k_pad, mode);
    return cudaGetLastError();
}

cudaError_t launch_strassen_input(const float* x, void* V_hi, void* V_lo, const StrassenGeom& g, int mode, cudaStream_t stream)
{
    const int Kh = g.Cin / 2;
    if (g.N / 2 > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((g.HW + 31) / 32), (unsigned)((g.k_pad + 31) / 32), (unsigned)(g.N / 2));
    strassen_input_kernel<<<grid, 256, 0, stream>>>(x, V_hi, V_lo, g, Kh, mode);
    return cudaGetLastError();
}

cudaError_t launch_strassen_output(const float* M, const float* bias, float* y, const StrassenGeom& g, int relu,
                                   cudaStream_t stream)
{
    const int Mh = g.Cout / 2;
    if (Mh > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((g.t_half + 127) / 128), (unsigned)Mh);
    strassen_output_kernel<<<grid, 128, 0, stream>>>(M, bias, y, g, Mh, relu);
    return cudaGetLastError();
}

}  // namespace mnnb
