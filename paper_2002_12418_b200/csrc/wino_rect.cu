// One-dimensional Winograd F(m, k) for 1 x k and k x 1 kernels (Section 4.2; Eq. 6 along one axis).
#include "wino_rect.h"

#include <cuda_bf16.h>

#include "wino_transforms.cuh"

namespace mnnb {

namespace {

using wino::store_operand;

struct RectMats {
    float Bt[kRectMaxAlpha * kRectMaxAlpha];
    float At[6 * kRectMaxAlpha];
    float G[kRectMaxAlpha * 7];
};

__global__ void rect_weights_kernel(const float* __restrict__ w, void* U_hi, void* U_lo, RectGeom g, int mode, RectMats mt)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long plane = (long long)g.Cout * g.cin_pad;
    if (gid >= plane) return;
    const int ci = (int)(gid % g.cin_pad), co = (int)(gid / g.cin_pad);
    float tap[7];
    for (int a = 0; a < g.k; ++a) tap[a] = ci < g.Cin ? w[((size_t)co * g.Cin + ci) * g.k + a] : 0.0f;
    for (int xi = 0; xi < g.alpha; ++xi) {
        float s = 0.0f;
        for (int a = 0; a < g.k; ++a) s = fmaf(mt.G[xi * g.k + a], tap[a], s);
        store_operand(U_hi, U_lo, (size_t)xi * plane + (size_t)gid, s, mode);
    }
}

// One CTA: 32 tiles x 32 channels.  Lanes run over tiles while x is read (neighbouring tiles are neighbours in
// memory along the width, or the same column of neighbouring pixels along the height) and over channels while V
// is written (channel-contiguous rows), with a transposition through shared memory in between.
__global__ void __launch_bounds__(256) rect_input_kernel(const float* __restrict__ x, void* V_hi, void* V_lo, RectGeom g, int mode,
                                                         RectMats mt)
{
    __shared__ float s[kRectMaxAlpha][32][33];
    const long long t0 = (long long)blockIdx.x * 32;
    const int c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    {
        const long long t = t0 + tx;
        const bool t_ok = t < g.tiles;
        // decode the tile: the line it lies on and its first input position along the long axis
        int n = 0, fixed = 0, start = 0;                    // fixed: input row (along_w) or input column
        if (t_ok) {
            if (g.along_w) {
                const int seg = (int)(t % g.n_seg);
                const long long r = t / g.n_seg;
                fixed = (int)(r % g.OH) - g.pad_h;
                n = (int)(r / g.OH);
                start = seg * g.m - g.pad_w;
            } else {
                fixed = (int)(t % g.OW) - g.pad_w;
                const long long r = t / g.OW;
                n = (int)(r / g.n_seg);
                start = (int)(r % g.n_seg) * g.m - g.pad_h;
            }
        }
        const int fixed_extent = g.along_w ? g.H : g.W, long_extent = g.along_w ? g.W : g.H;
        const bool line_ok = t_ok && fixed >= 0 && fixed < fixed_extent;
        for (int r = ty; r < 32; r += 8) {
            const int c = c0 + r;
            float d[kRectMaxAlpha];
            const float* base = x + ((size_t)n * g.Cin + (c < g.Cin ? c : 0)) * g.H * g.W;
#pragma unroll
            for (int j = 0; j < kRectMaxAlpha; ++j) {
                const int pos = start + j;
                const bool ok = j < g.alpha && line_ok && c < g.Cin && pos >= 0 && pos < long_extent;
                d[j] = ok ? __ldg(base + (g.along_w ? (size_t)fixed * g.W + pos : (size_t)pos * g.W + fixed)) : 0.0f;
            }
            for (int xi = 0; xi < g.alpha; ++xi) {
                float v = 0.0f;
#pragma unroll
                for (int j = 0; j < kRectMaxAlpha; ++j)
                    if (j < g.alpha) v = fmaf(mt.Bt[xi * g.alpha + j], d[j], v);
                s[xi][r][tx] = v;
            }
        }
    }
    __syncthreads();
    const int c = c0 + tx;
    if (c >= g.cin_pad) return;
    const size_t plane = (size_t)g.tiles * g.cin_pad;
    for (int r = ty; r < 32; r += 8) {
        const long long t = t0 + r;
        if (t >= g.tiles) break;
        for (int xi = 0; xi < g.alpha; ++xi)
            store_operand(V_hi, V_lo, (size_t)xi * plane + (size_t)t * g.cin_pad + c, s[xi][tx][r], mode);
    }
}

__global__ void __launch_bounds__(128) rect_output_kernel(const float* __restrict__ M, const float* __restrict__ bias,
                                                          float* __restrict__ y, RectGeom g, int relu, RectMats mt)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int co = blockIdx.y;
    if (t >= g.tiles) return;
    const size_t plane = (size_t)g.Cout * g.m_row_stride;
    const float* src = M + (size_t)co * g.m_row_stride + t;
    float mv[kRectMaxAlpha];
#pragma unroll
    for (int xi = 0; xi < kRectMaxAlpha; ++xi) mv[xi] = xi < g.alpha ? __ldcs(src + xi * plane) : 0.0f;
    const float b = bias ? __ldg(bias + co) : 0.0f;
    int n, oh, ow, step, limit;
    if (g.along_w) {
        const int seg = (int)(t % g.n_seg);
        const long long r = t / g.n_seg;
        oh = (int)(r % g.OH);
        n = (int)(r / g.OH);
        ow = seg * g.m;
        step = 1;
        limit = g.OW - ow;
    } else {
        ow = (int)(t % g.OW);
        const long long r = t / g.OW;
        n = (int)(r / g.n_seg);
        oh = (int)(r % g.n_seg) * g.m;
        step = g.OW;
        limit = g.OH - oh;
    }
    float* dst = y + (((size_t)n * g.Cout + co) * g.OH + oh) * g.OW + ow;
    for (int a = 0; a < g.m && a < limit; ++a) {
        float v = b;
#pragma unroll
        for (int xi = 0; xi < kRectMaxAlpha; ++xi)
            if (xi < g.alpha) v = fmaf(mt.At[a * g.alpha + xi], mv[xi], v);
        dst[(size_t)a * step] = relu ? fmaxf(v, 0.0f) : v;
    }
}

RectMats pack(const TransformMatrices& mats, const RectGeom& g)
{
    RectMats mt = {};
    for (int i = 0; i < g.alpha * g.alpha; ++i) mt.Bt[i] = mats.Bt[i];
    for (int i = 0; i < g.m * g.alpha; ++i) mt.At[i] = mats.At[i];
    for (int i = 0; i < g.alpha * g.k; ++i) mt.G[i] = mats.G[i];
    return mt;
}

bool geom_ok(const RectGeom& g) { return g.alpha <= kRectMaxAlpha && g.alpha == g.m + g.k - 1 && g.k <= 7 && g.m <= 6; }

}  // namespace

cudaError_t launch_rect_weights(const float* w, void* U_hi, void* U_lo, const RectGeom& g, int mode, const TransformMatrices& mats,
                                cudaStream_t stream)
{
    if (!geom_ok(g)) return cudaErrorInvalidValue;
    const long long total = (long long)g.Cout * g.cin_pad;
    rect_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(w, U_hi, U_lo, g, mode, pack(mats, g));
    return cudaGetLastError();
}

cudaError_t launch_rect_input(const float* x, void* V_hi, void* V_lo, const RectGeom& g, int mode, const TransformMatrices& mats,
                              cudaStream_t stream)
{
    if (!geom_ok(g) || (g.tiles + 31) / 32 > 2147483647ll) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((g.tiles + 31) / 32), (unsigned)((g.cin_pad + 31) / 32));
    rect_input_kernel<<<grid, 256, 0, stream>>>(x, V_hi, V_lo, g, mode, pack(mats, g));
    return cudaGetLastError();
}

cudaError_t launch_rect_output(const float* M, const float* bias, float* y, const RectGeom& g, int relu, const TransformMatrices& mats,
                               cudaStream_t stream)
{
    if (!geom_ok(g) || g.Cout > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((g.tiles + 127) / 128), (unsigned)g.Cout);
    rect_output_kernel<<<grid, 128, 0, stream>>>(M, bias, y, g, relu, pack(mats, g));
    return cudaGetLastError();
}

}  // namespace mnnb
