// Patch gather for the GEMM scheme and the direct ("sliding window", Section 3.2)
// convolution kernels.
#include <cuda_bf16.h>

#include "kernels.h"

namespace mnnb {

namespace {

__device__ __forceinline__ float round_tf32_g(float v)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

__device__ __forceinline__ void store_operand_g(void* hi, void* lo, size_t idx, float v, int mode)
{
    switch (mode) {
        case STORE_TF32:
            reinterpret_cast<float*>(hi)[idx] = round_tf32_g(v);
            break;
        case STORE_BF16:
            reinterpret_cast<__nv_bfloat16*>(hi)[idx] = __float2bfloat16_rn(v);
            break;
        case STORE_TF32_SPLIT: {
            const float h = round_tf32_g(v);
            reinterpret_cast<float*>(hi)[idx] = h;
            reinterpret_cast<float*>(lo)[idx] = round_tf32_g(v - h);
            break;
        }
        case STORE_BF16_SPLIT: {
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            reinterpret_cast<__nv_bfloat16*>(hi)[idx] = h;
            reinterpret_cast<__nv_bfloat16*>(lo)[idx] = __float2bfloat16_rn(v - __bfloat162float(h));
            break;
        }
        default:
            reinterpret_cast<float*>(hi)[idx] = v;
            break;
    }
}

// Generic gather: a 32 x 32 (output position x patch element) block per CTA is read
// with the output position fastest (adjacent pixels of x), transposed through
// shared memory and written with the patch element fastest (rows of V).
__global__ void __launch_bounds__(256) gather_kernel(const float* __restrict__ x, void* V_hi, void* V_lo, GatherGeom g,
                                                     long long T, int mode)
{
    __shared__ float tile[32][33];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the previous kernel of the stream has completed
    const long long t0 = (long long)blockIdx.x * 32;
    const int kk0 = blockIdx.y * 32;
    const int Kd = g.Cin * g.k * g.k;
    const int lx = threadIdx.x & 31, ly = threadIdx.x >> 5;      // 32 x 8
    const int ohw = g.OH * g.OW;
    // read: lx walks output positions, ly (+8 per step) walks patch elements
    const long long t = t0 + lx;
    int n = 0, oh = 0, ow = 0;
    const bool t_ok = t < T;
    if (t_ok) {
        n = (int)(t / ohw);
        const int pix = (int)(t % ohw);
        oh = pix / g.OW;
        ow = pix % g.OW;
    }
    for (int r = ly; r < 32; r += 8) {
        const int kk = kk0 + r;
        float v = 0.0f;
        if (t_ok && kk < Kd) {
            const int ci = kk / (g.k * g.k), e = kk % (g.k * g.k);
            const int a = e / g.k, b = e % g.k;
            const int ih = oh * g.stride - g.pad + a * g.dil, iw = ow * g.stride - g.pad + b * g.dil;
            if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) v = __ldg(x + (((size_t)n * g.Cin + ci) * g.H + ih) * g.W + iw);
        }
        tile[r][lx] = v;
    }
    __syncthreads();
    // write: lx walks patch elements, ly walks output positions
    for (int r = ly; r < 32; r += 8) {
        const long long tt = t0 + r;
        const int kk = kk0 + lx;
        if (tt < T && kk < g.k_pad) store_operand_g(V_hi, V_lo, (size_t)tt * g.k_pad + kk, tile[lx][r], mode);
    }
}

// Generic direct convolution: one thread per output element.
__global__ void __launch_bounds__(256) direct_generic_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                             const float* __restrict__ bias, float* __restrict__ y,
                                                             DirectGeom g, long long total)
{
    const int cpg = g.Cin / g.groups, opg = g.Cout / g.groups;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        long long f = idx;
        const int ow = (int)(f % g.OW); f /= g.OW;
        const int oh = (int)(f % g.OH); f /= g.OH;
        const int co = (int)(f % g.Cout);
        const int n = (int)(f / g.Cout);
        const int grp = co / opg;
        float acc = bias ? __ldg(bias + co) : 0.0f;
        for (int c = 0; c < cpg; ++c) {
            const float* xp = x + ((size_t)n * g.Cin + grp * cpg + c) * g.H * g.W;
            const float* wp = w + ((size_t)co * cpg + c) * g.k * g.k;
            for (int a = 0; a < g.k; ++a) {
                const int ih = oh * g.stride - g.pad + a * g.dil;
                if (ih < 0 || ih >= g.H) continue;
                for (int b = 0; b < g.k; ++b) {
                    const int iw = ow * g.stride - g.pad + b * g.dil;
                    if (iw < 0 || iw >= g.W) continue;
                    acc = fmaf(__ldg(wp + a * g.k + b), __ldg(xp + (size_t)ih * g.W + iw), acc);
                }
            }
        }
        y[idx] = g.relu ? fmaxf(acc, 0.0f) : acc;
    }
}

// Depthwise 3x3 (groups = C, dilation 1, stride 1 or 2): one warp sweeps a 32-column
// strip of one channel plane downwards.  Each lane keeps the three input rows of its
// output column group in registers; horizontal neighbours come from warp shuffles, so
// every input element is loaded once per strip.
template <int STRIDE>
__global__ void __launch_bounds__(128) depthwise3x3_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                           const float* __restrict__ bias, float* __restrict__ y,
                                                           DirectGeom g, int strips, long long n_units)
{
    const int lane = threadIdx.x & 31;
    const long long unit = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (plane, strip)
    if (unit >= n_units) return;
    const long long plane = unit / strips;
    const int strip = (int)(unit % strips);
    const int c = (int)(plane % g.Cout);
    const float* xp = x + (size_t)plane * g.H * g.W;
    float* yp = y + (size_t)plane * g.OH * g.OW;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + (size_t)c * 9 + i);
    const float b = bias ? __ldg(bias + c) : 0.0f;

    // Lane l produces output column ow = strip*30 + l - 1 + ... for stride 1 we let the 32 lanes
    // hold 32 input columns iw0 + l and produce outputs from the 30 interior lanes.
    if (STRIDE == 1) {
        const int iw = strip * 30 - g.pad + lane;           // input column held by this lane
        const int ow = iw - 1 + g.pad;                      // output whose centre tap is this column (pad = 1 -> ow = iw)
        const bool col_ok = iw >= 0 && iw < g.W;
        const bool out_ok = lane >= 1 && lane <= 30 && ow >= 0 && ow < g.OW;
        float r0 = 0.0f, r1 = 0.0f, r2;
        // rows: output row oh uses input rows oh - pad + {0,1,2}
        int ih = -g.pad;
        r0 = (col_ok && ih >= 0 && ih < g.H) ? __ldg(xp + (size_t)ih * g.W + iw) : 0.0f;
        ++ih;
        r1 = (col_ok && ih >= 0 && ih < g.H) ? __ldg(xp + (size_t)ih * g.W + iw) : 0.0f;
        for (int oh = 0; oh < g.OH; ++oh) {
            ih = oh - g.pad + 2;
            r2 = (col_ok && ih >= 0 && ih < g.H) ? __ldg(xp + (size_t)ih * g.W + iw) : 0.0f;
            float acc = b;
            const float l0 = __shfl_up_sync(0xffffffffu, r0, 1), l1 = __shfl_up_sync(0xffffffffu, r1, 1),
                        l2 = __shfl_up_sync(0xffffffffu, r2, 1);
            const float q0 = __shfl_down_sync(0xffffffffu, r0, 1), q1 = __shfl_down_sync(0xffffffffu, r1, 1),
                        q2 = __shfl_down_sync(0xffffffffu, r2, 1);
            acc = fmaf(wk[0], l0, acc); acc = fmaf(wk[1], r0, acc); acc = fmaf(wk[2], q0, acc);
            acc = fmaf(wk[3], l1, acc); acc = fmaf(wk[4], r1, acc); acc = fmaf(wk[5], q1, acc);
            acc = fmaf(wk[6], l2, acc); acc = fmaf(wk[7], r2, acc); acc = fmaf(wk[8], q2, acc);
            if (out_ok) yp[(size_t)oh * g.OW + ow] = g.relu ? fmaxf(acc, 0.0f) : acc;
            r0 = r1;
            r1 = r2;
        }
    } else {
        // stride 2: lane l produces output column ow = strip*32 + l and needs input columns 2*ow - pad + {0,1,2};
        // it loads the pair (2*ow - pad, 2*ow - pad + 1) and takes the third from the next lane.
        const int ow = strip * 32 + lane;
        const int iw0 = 2 * ow - g.pad;
        const bool out_ok = ow < g.OW;
        const bool c0_ok = iw0 >= 0 && iw0 < g.W, c1_ok = iw0 + 1 >= 0 && iw0 + 1 < g.W;
        // the last lane has no right neighbour: it loads its third column itself
        const int iw2 = iw0 + 2;
        const bool c2_ok = iw2 >= 0 && iw2 < g.W;
        for (int oh = 0; oh < g.OH; ++oh) {
            float acc = b;
#pragma unroll
            for (int a = 0; a < 3; ++a) {
                const int ih = 2 * oh - g.pad + a;
                const bool row_ok = ih >= 0 && ih < g.H;
                const float* rowp = xp + (size_t)(row_ok ? ih : 0) * g.W;
                const float v0 = (row_ok && c0_ok) ? __ldg(rowp + iw0) : 0.0f;
                const float v1 = (row_ok && c1_ok) ? __ldg(rowp + iw0 + 1) : 0.0f;
                float v2 = __shfl_down_sync(0xffffffffu, v0, 1);
                if (lane == 31) v2 = (row_ok && c2_ok) ? __ldg(rowp + iw2) : 0.0f;
                acc = fmaf(wk[a * 3 + 0], v0, acc);
                acc = fmaf(wk[a * 3 + 1], v1, acc);
                acc = fmaf(wk[a * 3 + 2], v2, acc);
            }
            if (out_ok) yp[(size_t)oh * g.OW + ow] = g.relu ? fmaxf(acc, 0.0f) : acc;
        }
    }
}

}  // namespace

cudaError_t launch_gather(const float* x, void* V_hi, void* V_lo, const GatherGeom& g, int mode, cudaStream_t stream)
{
    const long long T = (long long)g.N * g.OH * g.OW;
    if (T <= 0) return cudaSuccess;
    const long long bx = (T + 31) / 32;
    const int by = (g.k_pad + 31) / 32;
    if (bx > 2147483647ll || by > 65535) return cudaErrorInvalidValue;
    return launch_overlapped(gather_kernel, dim3((unsigned)bx, (unsigned)by), dim3(256), 0, stream, x, V_hi, V_lo, g, T, mode);
}

cudaError_t launch_direct(const float* x, const float* w, const float* bias, float* y, const DirectGeom& g,
                          cudaStream_t stream)
{
    const long long total = (long long)g.N * g.Cout * g.OH * g.OW;
    if (total <= 0) return cudaSuccess;
    const bool depthwise3 = g.groups == g.Cin && g.Cin == g.Cout && g.k == 3 && g.dil == 1 && g.pad == 1 &&
                            (g.stride == 1 || g.stride == 2);
    if (depthwise3) {
        const long long planes = (long long)g.N * g.Cout;
        const int strips = g.stride == 1 ? (g.OW + 29) / 30 : (g.OW + 31) / 32;
        const long long units = planes * strips;
        const long long blocks = (units + 3) / 4;
        if (blocks > 2147483647ll) return cudaErrorInvalidValue;
        if (g.stride == 1)
            depthwise3x3_kernel<1><<<(unsigned)blocks, 128, 0, stream>>>(x, w, bias, y, g, strips, units);
        else
            depthwise3x3_kernel<2><<<(unsigned)blocks, 128, 0, stream>>>(x, w, bias, y, g, strips, units);
        return cudaGetLastError();
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148ll * 64) blocks = 148ll * 64;
    direct_generic_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, w, bias, y, g, total);
    return cudaGetLastError();
}

}  // namespace mnnb
