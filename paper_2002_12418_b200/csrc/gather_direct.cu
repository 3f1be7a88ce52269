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

// Four consecutive elements of a row of V (idx a multiple of 4) in the operand format of MODE.
template <int MODE>
__device__ __forceinline__ void store_quad_g(void* V_hi, void* V_lo, size_t idx, const float (&v)[4])
{
    if (MODE == STORE_BF16 || MODE == STORE_BF16_SPLIT) {
        __nv_bfloat162 h01 = __floats2bfloat162_rn(v[0], v[1]), h23 = __floats2bfloat162_rn(v[2], v[3]);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&h01);
        pk.y = *reinterpret_cast<uint32_t*>(&h23);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(V_hi) + idx) = pk;
        if (MODE == STORE_BF16_SPLIT) {
            const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
            __nv_bfloat162 l01 = __floats2bfloat162_rn(v[0] - f01.x, v[1] - f01.y),
                           l23 = __floats2bfloat162_rn(v[2] - f23.x, v[3] - f23.y);
            pk.x = *reinterpret_cast<uint32_t*>(&l01);
            pk.y = *reinterpret_cast<uint32_t*>(&l23);
            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(V_lo) + idx) = pk;
        }
    } else if (MODE == STORE_FP32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(V_hi) + idx) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
        float h[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) h[e] = round_tf32_g(v[e]);
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(V_hi) + idx) = make_float4(h[0], h[1], h[2], h[3]);
        if (MODE == STORE_TF32_SPLIT)
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(V_lo) + idx) =
                make_float4(round_tf32_g(v[0] - h[0]), round_tf32_g(v[1] - h[1]), round_tf32_g(v[2] - h[2]),
                            round_tf32_g(v[3] - h[3]));
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

// 1 x 1, stride 1, no padding: the gather is a transposition of each image from [channel][pixel] to
// [pixel][channel] with rounding.  A CTA moves a 64 x 64 block through shared memory: 128-bit loads along
// the pixels, 128-bit (fp32 containers) or 64-bit (bf16) stores along the channels.  Needs H * W % 4 == 0.
template <int MODE>
__global__ void __launch_bounds__(256) gather_1x1_kernel(const float* __restrict__ x, void* V_hi, void* V_lo, int Cin, int hw,
                                                         int k_pad)
{
    __shared__ float tile[64][65];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int p0 = blockIdx.x * 64, c0 = blockIdx.y * 64, n = blockIdx.z;
    const float* xn = x + (size_t)n * Cin * hw;
    {
        const int pv = (threadIdx.x & 15) * 4, cr = threadIdx.x >> 4;      // 16 vectors of 4 pixels x 16 channels
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = cr + 16 * i;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c0 + c < Cin && p0 + pv < hw) v = __ldg(reinterpret_cast<const float4*>(xn + (size_t)(c0 + c) * hw + p0 + pv));
            tile[c][pv] = v.x; tile[c][pv + 1] = v.y; tile[c][pv + 2] = v.z; tile[c][pv + 3] = v.w;
        }
    }
    __syncthreads();
    const int cv = (threadIdx.x & 15) * 4, pr = threadIdx.x >> 4;          // 16 vectors of 4 channels x 16 pixels
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = pr + 16 * i;
        if (p0 + p >= hw || c0 + cv >= k_pad) continue;
        const size_t idx = ((size_t)n * hw + p0 + p) * k_pad + c0 + cv;     // multiple of 4: k_pad is a multiple of 8
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = tile[cv + e][p];
        store_quad_g<MODE>(V_hi, V_lo, idx, v);
    }
}

// Staged gather for k > 1 layers.  A CTA owns a block of output positions of one image (rt rows x
// seg_w columns) and a slab of patch elements (slab_q groups of four, i.e. whole 16-byte
// pieces of the rows of V; 64 positions, or up to 256 where the rows of V are short).  It copies the input region those positions touch, for the channels of the slab,
// into shared memory row by row (coalesced, zero outside the image), builds two offset tables (patch element
// -> offset inside the region, position -> offset of its window's corner) and then writes V: eight lanes
// cover 128 contiguous bytes of one row of V, a warp four rows at a time.  An element is region[koff + poff]:
// no division or bounds test per element.
struct StagedGather {
    int seg_w, segs, rt, row_tiles, rh, rw, slab_q, kq_n;
};

template <int MODE>
__global__ void __launch_bounds__(256) gather_staged_kernel(const float* __restrict__ x, void* V_hi, void* V_lo, GatherGeom g,
                                                            StagedGather sg)
{
    extern __shared__ __align__(16) unsigned char gs_raw[];
    int* koff = reinterpret_cast<int*>(gs_raw);                 // [slab_q * 4], -1 = padding element
    int* poff = koff + sg.slab_q * 4;                           // [256], -1 = no such position
    float* region = reinterpret_cast<float*>(poff + 256);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k2 = g.k * g.k, Kd = g.Cin * k2;
    const int kq0 = blockIdx.y * sg.slab_q, kq1 = min(sg.kq_n, kq0 + sg.slab_q);
    const int kk0 = 4 * kq0, kk1 = min(4 * kq1, Kd);            // real patch elements of the slab
    const int ci_lo = kk0 / k2, ci_hi = kk1 > kk0 ? (kk1 - 1) / k2 : ci_lo - 1;
    int bx = blockIdx.x;
    const int seg = bx % sg.segs; bx /= sg.segs;
    const int rtile = bx % sg.row_tiles;
    const int n = bx / sg.row_tiles;
    const int oh0 = rtile * sg.rt, rows = min(sg.rt, g.OH - oh0);
    const int ow0 = seg * sg.seg_w, cols = min(sg.seg_w, g.OW - ow0);
    const int ih0 = oh0 * g.stride - g.pad, iw0 = ow0 * g.stride - g.pad;
    const int plane = sg.rh * sg.rw;

    for (int i = threadIdx.x; i < (kq1 - kq0) * 4; i += 256) {
        const int kk = kk0 + i;
        int o = -1;
        if (kk < Kd) {
            const int ci = kk / k2, e = kk - ci * k2, a = e / g.k, b = e - a * g.k;
            o = (ci - ci_lo) * plane + a * g.dil * sg.rw + b * g.dil;
        }
        koff[i] = o;
    }
    {
        const int r = threadIdx.x / sg.seg_w, c = threadIdx.x - r * sg.seg_w;
        poff[threadIdx.x] = (r < rows && c < cols) ? r * g.stride * sg.rw + c * g.stride : -1;
    }
    // region rows: a warp takes 32 / lw rows per pass, lw = the power of two that covers a row (at most 32)
    const int n_rows = (ci_hi - ci_lo + 1) * sg.rh;
    int lw = 32;
    while (lw > 1 && (lw >> 1) >= sg.rw) lw >>= 1;
    const int rows_per_pass = 32 / lw, sub = lane / lw, lc = lane - sub * lw;
#pragma unroll 4
    for (int row = warp * rows_per_pass + sub; row < n_rows; row += 8 * rows_per_pass) {
        const int ch = row / sg.rh, rh = row - ch * sg.rh;
        const int ci = ci_lo + ch, ih = ih0 + rh;
        const bool row_ok = ci < g.Cin && ih >= 0 && ih < g.H;
        const float* src = x + (((size_t)n * g.Cin + (row_ok ? ci : 0)) * g.H + (row_ok ? ih : 0)) * g.W;
        float* dst = region + (size_t)row * sg.rw;
        for (int c = lc; c < sg.rw; c += lw) {
            const int iw = iw0 + c;
            dst[c] = (row_ok && iw >= 0 && iw < g.W) ? __ldg(src + iw) : 0.0f;
        }
    }
    __syncthreads();

    const int kql = lane & 7, tl = lane >> 3;
    const int n_pos = sg.rt * sg.seg_w;                         // <= 256
    const int4* koff4 = reinterpret_cast<const int4*>(koff);
    for (int tb = warp * 4; tb < n_pos; tb += 32) {
        const int ti = tb + tl;
        const int po = ti < n_pos ? poff[ti] : -1;
        if (po < 0) continue;
        const int r = ti / sg.seg_w, c = ti - r * sg.seg_w;
        const size_t t = ((size_t)n * g.OH + oh0 + r) * g.OW + ow0 + c;
        for (int kq = kq0 + kql; kq < kq1; kq += 8) {
            const int4 ko = koff4[kq - kq0];
            float v[4];
            v[0] = ko.x < 0 ? 0.0f : region[ko.x + po];
            v[1] = ko.y < 0 ? 0.0f : region[ko.y + po];
            v[2] = ko.z < 0 ? 0.0f : region[ko.z + po];
            v[3] = ko.w < 0 ? 0.0f : region[ko.w + po];
            store_quad_g<MODE>(V_hi, V_lo, t * g.k_pad + 4 * (size_t)kq, v);
        }
    }
}

// Block shape of the staged gather for a layer; false when no slab of at least 8 groups fits the shared-memory budget.
bool plan_staged_gather(const GatherGeom& g, StagedGather* sg, size_t* smem)
{
    constexpr int kRegionFloats = 9216;                          // 36 KB
    // (1x1 strided layers would stage rows and columns they never use: the element-wise gather serves them)
    if (g.k_pad % 4 != 0 || g.k == 1) return false;
    const int parts = (g.OW + 63) / 64;
    sg->seg_w = (g.OW + parts - 1) / parts;
    sg->segs = (g.OW + sg->seg_w - 1) / sg->seg_w;
    // positions per CTA: enough for some tens of kilobytes of V per CTA when its rows are short
    const int max_pos = g.k_pad <= 64 ? 256 : (g.k_pad <= 128 ? 128 : 64);
    int rt = max_pos / sg->seg_w;
    if (rt < 1) rt = 1;
    if (rt > g.OH) rt = g.OH;
    sg->rt = rt;
    sg->row_tiles = (g.OH + rt - 1) / rt;
    sg->rh = (rt - 1) * g.stride + (g.k - 1) * g.dil + 1;
    sg->rw = (sg->seg_w - 1) * g.stride + (g.k - 1) * g.dil + 1;
    sg->kq_n = g.k_pad / 4;
    const int k2 = g.k * g.k;
    const long long plane = (long long)sg->rh * sg->rw;
    int best = 0;
    for (int q = 8; q <= 64; q += 8) {
        const int qq = q < sg->kq_n ? q : sg->kq_n;
        const long long chans = (4LL * qq + k2 - 2) / k2 + 1;    // channels a slab of qq groups can touch
        if (chans * plane <= kRegionFloats) best = qq;
        if (qq == sg->kq_n) break;
    }
    if (best == 0) return false;
    sg->slab_q = best;
    const long long chans = (4LL * best + k2 - 2) / k2 + 1;
    *smem = (size_t)best * 16 + 256 * 4 + (size_t)(chans * plane) * 4;
    return true;
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

// Layers with very few input channels (network stems: Cin <= 4, groups 1): one thread per output pixel.  The
// weights sit in shared memory as [tap][output channel], so the 32 output channels a thread accumulates at a
// time come from eight broadcast 128-bit loads per tap; the patch values are re-read per group of 32 channels
// from L1.  Stores are coalesced along the pixels.
constexpr int kStemThreads = 128;
constexpr int kStemCoChunk = 32;

__global__ void __launch_bounds__(kStemThreads) direct_stem_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                                   const float* __restrict__ bias, float* __restrict__ y,
                                                                   DirectGeom g, int co_pad)
{
    extern __shared__ __align__(16) float s_w[];              // [Cin * k * k][co_pad]
    const int taps = g.Cin * g.k * g.k;
    for (int i = threadIdx.x; i < taps * co_pad; i += kStemThreads) {
        const int tap = i / co_pad, co = i - tap * co_pad;
        s_w[i] = co < g.Cout ? __ldg(w + (size_t)co * taps + tap) : 0.0f;
    }
    __syncthreads();
    const int ohw = g.OH * g.OW;
    const int n = blockIdx.y;
    const int pix = blockIdx.x * kStemThreads + threadIdx.x;
    if (pix >= ohw) return;
    const int oh = pix / g.OW, ow = pix - oh * g.OW;
    const int ih0 = oh * g.stride - g.pad, iw0 = ow * g.stride - g.pad;
    const float* xn = x + (size_t)n * g.Cin * g.H * g.W;
    float* yn = y + (size_t)n * g.Cout * ohw + pix;
    for (int c0 = 0; c0 < g.Cout; c0 += kStemCoChunk) {
        float acc[kStemCoChunk];
#pragma unroll
        for (int j = 0; j < kStemCoChunk; ++j) acc[j] = (bias && c0 + j < g.Cout) ? __ldg(bias + c0 + j) : 0.0f;
        int tap = 0;
        for (int ci = 0; ci < g.Cin; ++ci) {
            const float* xc = xn + (size_t)ci * g.H * g.W;
            for (int a = 0; a < g.k; ++a) {
                const int ih = ih0 + a * g.dil;
                const bool row_ok = ih >= 0 && ih < g.H;
                for (int b = 0; b < g.k; ++b, ++tap) {
                    const int iw = iw0 + b * g.dil;
                    const float v = (row_ok && iw >= 0 && iw < g.W) ? __ldg(xc + (size_t)ih * g.W + iw) : 0.0f;
                    const float4* wp = reinterpret_cast<const float4*>(s_w + (size_t)tap * co_pad + c0);
#pragma unroll
                    for (int q = 0; q < kStemCoChunk / 4; ++q) {
                        const float4 w4 = wp[q];
                        acc[4 * q] = fmaf(w4.x, v, acc[4 * q]);
                        acc[4 * q + 1] = fmaf(w4.y, v, acc[4 * q + 1]);
                        acc[4 * q + 2] = fmaf(w4.z, v, acc[4 * q + 2]);
                        acc[4 * q + 3] = fmaf(w4.w, v, acc[4 * q + 3]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kStemCoChunk; ++j)
            if (c0 + j < g.Cout) yn[(size_t)(c0 + j) * ohw] = g.relu ? fmaxf(acc[j], 0.0f) : acc[j];
    }
}

// The same layer with its shape fixed at compile time (dilation 1): all CIN * K * K input values of a thread's
// PIX output pixels are requested before the first is used, and the multiply-adds run as packed pairs of fp32
// lanes (__ffma2_rn: two IEEE fused multiply-adds per instruction, the results of the scalar kernel bit for
// bit), with one shared-memory weight fetch serving all PIX pixels.
template <int CIN, int K, int STRIDE, int PIX>
__global__ void __launch_bounds__(kStemThreads) direct_stem_fixed_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                                         const float* __restrict__ bias, float* __restrict__ y,
                                                                         DirectGeom g, int co_pad)
{
    constexpr int TAPS = CIN * K * K;
    extern __shared__ __align__(16) float s_w[];              // [TAPS][co_pad]
    for (int i = threadIdx.x; i < TAPS * co_pad; i += kStemThreads) {
        const int tap = i / co_pad, co = i - tap * co_pad;
        s_w[i] = co < g.Cout ? __ldg(w + (size_t)co * TAPS + tap) : 0.0f;
    }
    __syncthreads();
    const int ohw = g.OH * g.OW;
    const int n = blockIdx.y;
    const int pix0 = blockIdx.x * (kStemThreads * PIX) + threadIdx.x;
    const float* xn = x + (size_t)n * CIN * g.H * g.W;
    float v[PIX][TAPS];
#pragma unroll
    for (int p = 0; p < PIX; ++p) {
        const int pix = pix0 + p * kStemThreads;
        const bool live = pix < ohw;
        const int oh = pix / g.OW, ow = pix - oh * g.OW;
        const int ih0 = oh * STRIDE - g.pad, iw0 = ow * STRIDE - g.pad;
#pragma unroll
        for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
            for (int a = 0; a < K; ++a)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int ih = ih0 + a, iw = iw0 + b;
                    const bool ok = live && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W;
                    v[p][(ci * K + a) * K + b] = ok ? __ldg(xn + ((size_t)ci * g.H + ih) * g.W + iw) : 0.0f;
                }
    }
    for (int c0 = 0; c0 < g.Cout; c0 += kStemCoChunk) {
        float2 acc[PIX][kStemCoChunk / 2];
#pragma unroll
        for (int j = 0; j < kStemCoChunk / 2; ++j) {
            const float b0 = (bias && c0 + 2 * j < g.Cout) ? __ldg(bias + c0 + 2 * j) : 0.0f;
            const float b1 = (bias && c0 + 2 * j + 1 < g.Cout) ? __ldg(bias + c0 + 2 * j + 1) : 0.0f;
#pragma unroll
            for (int p = 0; p < PIX; ++p) acc[p][j] = make_float2(b0, b1);
        }
#pragma unroll
        for (int tap = 0; tap < TAPS; ++tap) {
            const float4* wp = reinterpret_cast<const float4*>(s_w + (size_t)tap * co_pad + c0);
            float2 vv[PIX];
#pragma unroll
            for (int p = 0; p < PIX; ++p) vv[p] = make_float2(v[p][tap], v[p][tap]);
#pragma unroll
            for (int q = 0; q < kStemCoChunk / 4; ++q) {
                const float4 w4 = wp[q];
#pragma unroll
                for (int p = 0; p < PIX; ++p) {
                    acc[p][2 * q] = __ffma2_rn(make_float2(w4.x, w4.y), vv[p], acc[p][2 * q]);
                    acc[p][2 * q + 1] = __ffma2_rn(make_float2(w4.z, w4.w), vv[p], acc[p][2 * q + 1]);
                }
            }
        }
        const bool full = c0 + kStemCoChunk <= g.Cout;
#pragma unroll
        for (int p = 0; p < PIX; ++p) {
            const int pix = pix0 + p * kStemThreads;
            if (pix >= ohw) continue;
            float* yp = y + ((size_t)n * g.Cout + c0) * ohw + pix;
#pragma unroll
            for (int j = 0; j < kStemCoChunk / 2; ++j) {
                float lo = acc[p][j].x, hi = acc[p][j].y;
                if (g.relu) { lo = fmaxf(lo, 0.0f); hi = fmaxf(hi, 0.0f); }
                if (full || c0 + 2 * j < g.Cout) yp[(size_t)(2 * j) * ohw] = lo;
                if (full || c0 + 2 * j + 1 < g.Cout) yp[(size_t)(2 * j + 1) * ohw] = hi;
            }
        }
    }
}

// 3 -> Cout, 3x3, stride 2, padding 1 on planes with H even and W a multiple of 4 (the first layer of the
// ImageNet networks).  A thread owns a block of ROWS x 2 output pixels (ROWS = 2 when H is a multiple of 4):
// its (2 ROWS + 1) x 5 x 3 input values come from two aligned float2 loads and one scalar load per row, the two
// results of a channel and row leave as one float2 store, and only the row above the plane and the column
// left of it can fall outside.  One 16-byte weight fetch from shared memory feeds 2 ROWS packed multiply-adds
// (__ffma2_rn: two IEEE fused multiply-adds per instruction, bit for bit the scalar result).  Blocks walk
// over (image, group of 128 pixel blocks) units and stage the weights once.
constexpr int kPairCoChunk = 16;   // output channels per sweep over the 27 taps

template <bool RELU, int ROWS>
__global__ void __launch_bounds__(kStemThreads, ROWS == 1 ? 5 : 3)
direct_stem_s2_pair_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                           float* __restrict__ y, DirectGeom g, int co_pad, int groups, int n_units)
{
    constexpr int CIN = 3, K = 3, TAPS = CIN * K * K, NR = 2 * ROWS + 1, PIX = 2 * ROWS;
    extern __shared__ __align__(16) float s_w[];              // [TAPS][co_pad]
    for (int i = threadIdx.x; i < TAPS * co_pad; i += kStemThreads) {
        const int tap = i / co_pad, co = i - tap * co_pad;
        s_w[i] = co < g.Cout ? __ldg(w + (size_t)co * TAPS + tap) : 0.0f;
    }
    __syncthreads();
    const int ohw = g.OH * g.OW, half_w = g.OW >> 1, per_image = (g.OH / ROWS) * half_w;
    for (int unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
        const int n = unit / groups;
        const int pp = (unit - n * groups) * kStemThreads + threadIdx.x;
        if (pp >= per_image) continue;
        const int obr = pp / half_w;
        const int oh = obr * ROWS, ow = 2 * (pp - obr * half_w);
        const float* xn = x + (size_t)n * CIN * g.H * g.W + 2 * ow;
        float c[CIN][NR][5];
#pragma unroll
        for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                const int ih = 2 * oh - 1 + r;
                const bool row_ok = ih >= 0 && ih < g.H;
                const float* row = xn + ((size_t)ci * g.H + (row_ok ? ih : 0)) * g.W;
                const float2 m0 = __ldg(reinterpret_cast<const float2*>(row));
                const float2 m1 = __ldg(reinterpret_cast<const float2*>(row + 2));
                const float left = ow > 0 ? __ldg(row - 1) : 0.0f;
                c[ci][r][0] = row_ok ? left : 0.0f;
                c[ci][r][1] = row_ok ? m0.x : 0.0f;
                c[ci][r][2] = row_ok ? m0.y : 0.0f;
                c[ci][r][3] = row_ok ? m1.x : 0.0f;
                c[ci][r][4] = row_ok ? m1.y : 0.0f;
            }
        for (int c0 = 0; c0 < g.Cout; c0 += kPairCoChunk) {
            float2 acc[PIX][kPairCoChunk / 2];                 // pixel = 2 * row + column
#pragma unroll
            for (int j = 0; j < kPairCoChunk / 2; ++j) {
                const float b0 = (bias && c0 + 2 * j < g.Cout) ? __ldg(bias + c0 + 2 * j) : 0.0f;
                const float b1 = (bias && c0 + 2 * j + 1 < g.Cout) ? __ldg(bias + c0 + 2 * j + 1) : 0.0f;
#pragma unroll
                for (int p = 0; p < PIX; ++p) acc[p][j] = make_float2(b0, b1);
            }
            // the weights of tap t + 1 are fetched while tap t is multiplied
            const float4* wbase = reinterpret_cast<const float4*>(s_w + c0);
            const int wstep = co_pad >> 2;
            float4 wn[kPairCoChunk / 4];
#pragma unroll
            for (int q = 0; q < kPairCoChunk / 4; ++q) wn[q] = wbase[q];
#pragma unroll
            for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
                for (int a = 0; a < K; ++a)
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        const int tap = (ci * K + a) * K + b;
                        float4 wc[kPairCoChunk / 4];
#pragma unroll
                        for (int q = 0; q < kPairCoChunk / 4; ++q) wc[q] = wn[q];
                        if (tap + 1 < TAPS) {
#pragma unroll
                            for (int q = 0; q < kPairCoChunk / 4; ++q) wn[q] = wbase[(tap + 1) * wstep + q];
                        }
                        float2 v[PIX];
#pragma unroll
                        for (int p = 0; p < PIX; ++p) {
                            const float e = c[ci][2 * (p >> 1) + a][b + 2 * (p & 1)];
                            v[p] = make_float2(e, e);
                        }
#pragma unroll
                        for (int q = 0; q < kPairCoChunk / 4; ++q) {
                            const float4 w4 = wc[q];
#pragma unroll
                            for (int p = 0; p < PIX; ++p) {
                                acc[p][2 * q] = __ffma2_rn(make_float2(w4.x, w4.y), v[p], acc[p][2 * q]);
                                acc[p][2 * q + 1] = __ffma2_rn(make_float2(w4.z, w4.w), v[p], acc[p][2 * q + 1]);
                            }
                        }
                    }
            const bool full = c0 + kPairCoChunk <= g.Cout;
#pragma unroll
            for (int rr = 0; rr < ROWS; ++rr) {
                float* yp = y + ((size_t)n * g.Cout + c0) * ohw + (size_t)(oh + rr) * g.OW + ow;
#pragma unroll
                for (int j = 0; j < kPairCoChunk / 2; ++j) {
                    float2 e = make_float2(acc[2 * rr][j].x, acc[2 * rr + 1][j].x);
                    float2 o = make_float2(acc[2 * rr][j].y, acc[2 * rr + 1][j].y);
                    if (RELU) {
                        e.x = fmaxf(e.x, 0.0f); e.y = fmaxf(e.y, 0.0f);
                        o.x = fmaxf(o.x, 0.0f); o.y = fmaxf(o.y, 0.0f);
                    }
                    if (full || c0 + 2 * j < g.Cout) *reinterpret_cast<float2*>(yp + (size_t)(2 * j) * ohw) = e;
                    if (full || c0 + 2 * j + 1 < g.Cout) *reinterpret_cast<float2*>(yp + (size_t)(2 * j + 1) * ohw) = o;
                }
            }
        }
    }
}

// Depthwise 3x3 (groups = C, dilation 1, padding 1, stride 1 or 2): one warp sweeps a strip of one channel
// plane downwards over a band of output rows.  A lane holds its column of the three input rows that an output
// row needs; horizontal neighbours come from warp shuffles, so every input element is loaded once per strip
// (plus two halo rows per band).  Four input rows are requested before any of them is used, which keeps
// enough loads in flight for the kernel to follow the memory system rather than its latency.
constexpr int kDwBandRows = 32;   // output rows per unit

// SW = lanes per plane segment (32, 16 or 8): narrow planes put 2 or 4 channel planes side by side in a warp.
template <int STRIDE, int SW>
__global__ void __launch_bounds__(128) depthwise3x3_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                           const float* __restrict__ bias, float* __restrict__ y,
                                                           DirectGeom g, int strips, int bands, long long n_planes,
                                                           long long n_units)
{
    constexpr int PPW = 32 / SW;                      // planes per warp
    const int lane = threadIdx.x & 31, ls = lane % SW, seg = lane / SW;
    const long long unit = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (plane group, band, strip)
    if (unit >= n_units) return;
    const int strip = (int)(unit % strips);
    const long long rest = unit / strips;
    const int band = (int)(rest % bands);
    const long long plane = (rest / bands) * PPW + seg;
    const bool plane_ok = plane < n_planes;
    const int c = (int)((plane_ok ? plane : 0) % g.Cout);
    const float* xp = x + (size_t)(plane_ok ? plane : 0) * g.H * g.W;
    float* yp = y + (size_t)(plane_ok ? plane : 0) * g.OH * g.OW;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + (size_t)c * 9 + i);
    const float b = bias ? __ldg(bias + c) : 0.0f;
    const int oh0 = band * kDwBandRows, oh1 = min(g.OH, oh0 + kDwBandRows);
    const unsigned full = 0xffffffffu;

    if (STRIDE == 1) {
        // a segment holds input columns strip * (SW - 2) - 1 + ls; lanes 1 .. SW - 2 produce outputs, and so does
        // the last lane when its right neighbour lies beyond the image (it is zero padding then)
        const int iw = strip * (SW - 2) - 1 + ls;
        const int ow = iw;
        const bool col_ok = plane_ok && iw >= 0 && iw < g.W;
        const bool last_edge = ls == SW - 1 && iw + 1 >= g.W;
        const bool out_ok = col_ok && ls >= 1 && (ls <= SW - 2 || last_edge) && ow < g.OW;
        auto row = [&](int ih) { return (col_ok && ih >= 0 && ih < g.H) ? __ldg(xp + (size_t)ih * g.W + iw) : 0.0f; };
        auto right = [&](float v) {
            const float n = __shfl_down_sync(full, v, 1, SW);
            return ls == SW - 1 ? 0.0f : n;
        };
        // per input row: the lane's own value and its left / right neighbours (shuffled once, when the row arrives)
        float r0 = row(oh0 - 1), r1 = row(oh0);
        float l0 = __shfl_up_sync(full, r0, 1, SW), q0 = right(r0);
        float l1 = __shfl_up_sync(full, r1, 1, SW), q1 = right(r1);
        for (int oh = oh0; oh < oh1; oh += 4) {
            float nx[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) nx[k] = row(oh + k + 1);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // (rows past the band are computed and not stored, so that the row registers rotate unconditionally)
                const float r2 = nx[k];
                const float l2 = __shfl_up_sync(full, r2, 1, SW), q2 = right(r2);
                float acc = b;
                acc = fmaf(wk[0], l0, acc); acc = fmaf(wk[1], r0, acc); acc = fmaf(wk[2], q0, acc);
                acc = fmaf(wk[3], l1, acc); acc = fmaf(wk[4], r1, acc); acc = fmaf(wk[5], q1, acc);
                acc = fmaf(wk[6], l2, acc); acc = fmaf(wk[7], r2, acc); acc = fmaf(wk[8], q2, acc);
                if (out_ok && oh + k < oh1) yp[(size_t)(oh + k) * g.OW + ow] = g.relu ? fmaxf(acc, 0.0f) : acc;
                l0 = l1; r0 = r1; q0 = q1;
                l1 = l2; r1 = r2; q1 = q2;
            }
        }
    } else {
        // lane ls of a segment produces output column ow = strip * SW + ls from input columns 2 ow - 1 + {0, 1, 2}:
        // it loads the first two and takes the third from the next lane (the segment's last lane loads its own)
        const int ow = strip * SW + ls;
        const int iw0 = 2 * ow - 1;
        const bool out_ok = plane_ok && ow < g.OW;
        const bool c0_ok = plane_ok && iw0 >= 0 && iw0 < g.W, c1_ok = plane_ok && iw0 + 1 < g.W,
                   c2_ok = plane_ok && ls == SW - 1 && iw0 + 2 < g.W;
        struct Row { float v0, v1, v2; };
        auto load = [&](int ih, Row& r) {
            const bool ok = ih >= 0 && ih < g.H;
            const float* p = xp + (size_t)(ok ? ih : 0) * g.W + iw0;
            r.v0 = (ok && c0_ok) ? __ldg(p) : 0.0f;
            r.v1 = (ok && c1_ok) ? __ldg(p + 1) : 0.0f;
            r.v2 = (ok && c2_ok) ? __ldg(p + 2) : 0.0f;
        };
        auto third = [&](Row& r) {
            const float n = __shfl_down_sync(full, r.v0, 1, SW);
            if (ls != SW - 1) r.v2 = n;
        };
        auto out = [&](int oh, const Row& a, const Row& m, const Row& z) {
            float acc = b;
            acc = fmaf(wk[0], a.v0, acc); acc = fmaf(wk[1], a.v1, acc); acc = fmaf(wk[2], a.v2, acc);
            acc = fmaf(wk[3], m.v0, acc); acc = fmaf(wk[4], m.v1, acc); acc = fmaf(wk[5], m.v2, acc);
            acc = fmaf(wk[6], z.v0, acc); acc = fmaf(wk[7], z.v1, acc); acc = fmaf(wk[8], z.v2, acc);
            if (out_ok) yp[(size_t)oh * g.OW + ow] = g.relu ? fmaxf(acc, 0.0f) : acc;
        };
        Row prev;
        load(2 * oh0 - 1, prev);
        third(prev);
        for (int oh = oh0; oh < oh1; oh += 2) {
            Row ra, rb, rc, rd;                       // input rows 2 oh .. 2 oh + 3, all requested before use
            load(2 * oh, ra);
            load(2 * oh + 1, rb);
            load(2 * oh + 2, rc);
            load(2 * oh + 3, rd);
            third(ra); third(rb); third(rc); third(rd);
            out(oh, prev, ra, rb);
            if (oh + 1 < oh1) out(oh + 1, rb, rc, rd);
            prev = rd;
        }
    }
}

// The same sweep for even image widths, with VIN = 2 or 4 input columns per lane (W a multiple of VIN): rows are
// read and written with aligned 64- or 128-bit accesses, a warp keeps four whole rows of up to 512 bytes in
// flight, and a lane needs one value from its left neighbour per row (and one from its right neighbour at
// stride 1).  A lane holds input columns icol0 + [0, VIN) of its plane and produces VIN outputs (stride 1) or
// VIN / 2 (stride 2).  Planes no wider than SW * VIN take one strip with every lane productive; wider ones are
// cut into strips that overlap by one lane on the left (and one on the right at stride 1) whose columns the
// neighbouring strip produces.
template <int VIN>
struct DwRow {
    float e[VIN + 2];      // e[0] left neighbour, e[1 .. VIN] own columns, e[VIN + 1] right neighbour (stride 1)
};

template <int VIN>
__device__ __forceinline__ void dw_load_row(const float* __restrict__ p, bool ok, DwRow<VIN>& r)
{
    if (VIN == 4) {
        const float4 v = ok ? __ldg(reinterpret_cast<const float4*>(p)) : make_float4(0.f, 0.f, 0.f, 0.f);
        r.e[1] = v.x; r.e[2] = v.y; r.e[3] = v.z; r.e[VIN] = v.w;
    } else {
        const float2 v = ok ? __ldg(reinterpret_cast<const float2*>(p)) : make_float2(0.f, 0.f);
        r.e[1] = v.x; r.e[VIN] = v.y;
    }
}

// HMAX > 0 (planes of at most HMAX rows): every row of the plane is requested before the first is used, one
// trip to memory per warp instead of one per four rows, which is what short planes (14 x 14, 7 x 7) are bound by.
template <int STRIDE, int SW, int VIN, int HMAX = 0>
__global__ void __launch_bounds__(128) depthwise3x3_vec_kernel(const float* __restrict__ x, const float* __restrict__ w,
                                                               const float* __restrict__ bias, float* __restrict__ y,
                                                               DirectGeom g, int strips, int bands, long long n_planes,
                                                               long long n_units)
{
    constexpr int PPW = 32 / SW;                      // planes per warp
    constexpr int VOUT = STRIDE == 1 ? VIN : VIN / 2;
    const int lane = threadIdx.x & 31, ls = lane % SW, seg = lane / SW;
    // (plane group, band, strip) in 32-bit arithmetic: the launcher refuses more than 2^31 - 1 units
    const unsigned unit = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if ((long long)unit >= n_units) return;
    const int strip = (int)(unit % (unsigned)strips);
    const unsigned rest = unit / (unsigned)strips;
    const int band = (int)(rest % (unsigned)bands);
    const unsigned plane = (rest / (unsigned)bands) * PPW + seg;
    const bool plane_ok = (long long)plane < n_planes;
    const int c = (int)((plane_ok ? plane : 0u) % (unsigned)g.Cout);
    const float* xp = x + (size_t)(plane_ok ? plane : 0) * g.H * g.W;
    float* yp = y + (size_t)(plane_ok ? plane : 0) * g.OH * g.OW;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + (size_t)c * 9 + i);
    const float b = bias ? __ldg(bias + c) : 0.0f;
    const int oh0 = band * kDwBandRows, oh1 = min(g.OH, oh0 + kDwBandRows);
    const unsigned full = 0xffffffffu;

    // columns of this lane
    const int lanes_per_strip = STRIDE == 1 ? SW - 2 : SW - 1;            // productive lanes of an overlapping strip
    const int in_base = strips == 1 ? 0 : strip * lanes_per_strip * VIN - VIN;
    const int icol0 = in_base + ls * VIN;
    const bool col_ok = plane_ok && icol0 >= 0 && icol0 < g.W;            // the whole vector lies inside or outside
    const bool owns = col_ok && (ls >= 1 || strips == 1) && (STRIDE == 2 || ls <= SW - 2 || strip == strips - 1);
    const int ocol0 = STRIDE == 1 ? icol0 : icol0 / 2;
    // Rows are addressed by running pointers (one 32-bit multiply per loaded row, none per stored row); the row
    // registers rotate unconditionally and only the store of a row past the band is suppressed, so that the
    // unrolled loop needs no register moves.
    const float* xcol = xp + (col_ok ? icol0 : 0);
    const int Hd = g.H, Wd = g.W, OWd = g.OW;
    auto load = [&](int ih, DwRow<VIN>& r) {
        const bool ok = col_ok && (unsigned)ih < (unsigned)Hd;
        dw_load_row<VIN>(xcol + (ok ? ih * Wd : 0), ok, r);
    };
    auto edges = [&](DwRow<VIN>& r) {                                      // neighbours' border values
        const float l = __shfl_up_sync(full, r.e[VIN], 1, SW);
        r.e[0] = ls == 0 ? 0.0f : l;
        if (STRIDE == 1) {
            const float q = __shfl_down_sync(full, r.e[1], 1, SW);
            r.e[VIN + 1] = ls == SW - 1 ? 0.0f : q;
        }
    };
    const bool relu = g.relu != 0;
    auto out = [&](float* q, bool store, const DwRow<VIN>& a, const DwRow<VIN>& m, const DwRow<VIN>& z) {
        float acc[VOUT];
#pragma unroll
        for (int j = 0; j < VOUT; ++j) {
            float v = b;
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                v = fmaf(wk[t], a.e[STRIDE * j + t], v);
                v = fmaf(wk[3 + t], m.e[STRIDE * j + t], v);
                v = fmaf(wk[6 + t], z.e[STRIDE * j + t], v);
            }
            acc[j] = v;
        }
        if (relu) {
#pragma unroll
            for (int j = 0; j < VOUT; ++j) acc[j] = fmaxf(acc[j], 0.0f);
        }
        if (store) {
            if (VOUT == 4) *reinterpret_cast<float4*>(q) = make_float4(acc[0], acc[1], acc[2], acc[VOUT - 1]);
            else if (VOUT == 2) *reinterpret_cast<float2*>(q) = make_float2(acc[0], acc[VOUT - 1]);
            else *q = acc[0];
        }
    };
    float* yrow = yp + (owns ? oh0 * OWd + ocol0 : 0);                     // output row oh0 of this lane's columns

    if constexpr (HMAX > 0) {
        DwRow<VIN> rows[HMAX + 2];                    // rows[i] = input row i - 1; rows outside the plane are zero
#pragma unroll
        for (int i = 0; i < HMAX + 2; ++i) load(i - 1, rows[i]);
#pragma unroll
        for (int i = 0; i < HMAX + 2; ++i) edges(rows[i]);
#pragma unroll
        for (int k = 0; k < (STRIDE == 1 ? HMAX : (HMAX + 1) / 2); ++k)
            out(yrow + k * OWd, owns && k < oh1, rows[STRIDE * k], rows[STRIDE * k + 1], rows[STRIDE * k + 2]);
        return;
    }
    if (STRIDE == 1) {
        DwRow<VIN> r0, r1;
        load(oh0 - 1, r0);
        load(oh0, r1);
        edges(r0);
        edges(r1);
        for (int oh = oh0; oh < oh1; oh += 4) {
            DwRow<VIN> nx[4];                         // input rows oh + 1 .. oh + 4, all requested before use
#pragma unroll
            for (int k = 0; k < 4; ++k) load(oh + k + 1, nx[k]);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                edges(nx[k]);
                out(yrow + k * OWd, owns && oh + k < oh1, r0, r1, nx[k]);
                r0 = r1;
                r1 = nx[k];
            }
            yrow += 4 * OWd;
        }
    } else {
        DwRow<VIN> prev;
        load(2 * oh0 - 1, prev);
        edges(prev);
        for (int oh = oh0; oh < oh1; oh += 2) {
            DwRow<VIN> ra, rb, rc, rd;                // input rows 2 oh .. 2 oh + 3, all requested before use
            load(2 * oh, ra);
            load(2 * oh + 1, rb);
            load(2 * oh + 2, rc);
            load(2 * oh + 3, rd);
            edges(ra); edges(rb); edges(rc); edges(rd);
            out(yrow, owns, prev, ra, rb);
            out(yrow + OWd, owns && oh + 1 < oh1, rb, rc, rd);
            prev = rd;
            yrow += 2 * OWd;
        }
    }
}

}  // namespace

cudaError_t launch_gather(const float* x, void* V_hi, void* V_lo, const GatherGeom& g, int mode, cudaStream_t stream)
{
    const long long T = (long long)g.N * g.OH * g.OW;
    if (T <= 0) return cudaSuccess;
    const int hw = g.H * g.W;
    if (g.k == 1 && g.stride == 1 && g.pad == 0 && hw % 4 == 0 && g.N <= 65535 && (g.k_pad + 63) / 64 <= 65535) {
        const dim3 grid((unsigned)((hw + 63) / 64), (unsigned)((g.k_pad + 63) / 64), (unsigned)g.N);
        switch (mode) {
            case STORE_TF32: return launch_overlapped(gather_1x1_kernel<STORE_TF32>, grid, dim3(256), 0, stream, x, V_hi, V_lo, g.Cin, hw, g.k_pad);
            case STORE_BF16: return launch_overlapped(gather_1x1_kernel<STORE_BF16>, grid, dim3(256), 0, stream, x, V_hi, V_lo, g.Cin, hw, g.k_pad);
            case STORE_TF32_SPLIT: return launch_overlapped(gather_1x1_kernel<STORE_TF32_SPLIT>, grid, dim3(256), 0, stream, x, V_hi, V_lo, g.Cin, hw, g.k_pad);
            case STORE_BF16_SPLIT: return launch_overlapped(gather_1x1_kernel<STORE_BF16_SPLIT>, grid, dim3(256), 0, stream, x, V_hi, V_lo, g.Cin, hw, g.k_pad);
            default: return launch_overlapped(gather_1x1_kernel<STORE_FP32>, grid, dim3(256), 0, stream, x, V_hi, V_lo, g.Cin, hw, g.k_pad);
        }
    }
    {
        StagedGather sg;
        size_t smem = 0;
        if (plan_staged_gather(g, &sg, &smem)) {
            const long long gx = (long long)g.N * sg.row_tiles * sg.segs;
            const int gy = (sg.kq_n + sg.slab_q - 1) / sg.slab_q;
            if (gx <= 2147483647ll && gy <= 65535 && smem <= 48 * 1024) {
                const dim3 grid((unsigned)gx, (unsigned)gy);
                switch (mode) {
                    case STORE_TF32: return launch_overlapped(gather_staged_kernel<STORE_TF32>, grid, dim3(256), smem, stream, x, V_hi, V_lo, g, sg);
                    case STORE_BF16: return launch_overlapped(gather_staged_kernel<STORE_BF16>, grid, dim3(256), smem, stream, x, V_hi, V_lo, g, sg);
                    case STORE_TF32_SPLIT: return launch_overlapped(gather_staged_kernel<STORE_TF32_SPLIT>, grid, dim3(256), smem, stream, x, V_hi, V_lo, g, sg);
                    case STORE_BF16_SPLIT: return launch_overlapped(gather_staged_kernel<STORE_BF16_SPLIT>, grid, dim3(256), smem, stream, x, V_hi, V_lo, g, sg);
                    default: return launch_overlapped(gather_staged_kernel<STORE_FP32>, grid, dim3(256), smem, stream, x, V_hi, V_lo, g, sg);
                }
            }
        }
    }
    const long long bx = (T + 31) / 32;
    const int by = (g.k_pad + 31) / 32;
    if (bx > 2147483647ll || by > 65535) return cudaErrorInvalidValue;
    return launch_overlapped(gather_kernel, dim3((unsigned)bx, (unsigned)by), dim3(256), 0, stream, x, V_hi, V_lo, g, T, mode);
}

bool direct_stem_applies(const DirectGeom& g)
{
    const long long smem = (long long)g.Cin * g.k * g.k * ((g.Cout + 31) / 32 * 32) * 4;
    return g.groups == 1 && g.Cin <= 4 && g.N <= 65535 && smem <= 160 * 1024;
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
        const int bands = (g.OH + kDwBandRows - 1) / kDwBandRows;
        if (g.W % 2 == 0) {
            // even widths: 2 or 4 columns per lane, the narrowest segment that holds a row, else 32-lane strips
            const int vin = g.W % 4 == 0 ? 4 : 2;
            const int need = g.W / vin;
            const int sw = need <= 8 ? 8 : (need <= 16 ? 16 : 32);
            const int per_strip = (g.stride == 1 ? 30 : 31) * vin;
            const int strips = need <= 32 ? 1 : (g.W + per_strip - 1) / per_strip;
            const long long groups = (planes + 32 / sw - 1) / (32 / sw);
            const long long units = groups * strips * bands;
            const long long blocks = (units + 3) / 4;
            if (units > 2147483647ll - 4) return cudaErrorInvalidValue;
            // short planes held whole in registers: up to 16 rows with 2 columns per lane, up to 8 with 4
            if (strips == 1 && sw == 8 && g.H <= (vin == 2 ? 16 : 8)) {
#define MNNB_DWS_LAUNCH(ST, VI, HM) depthwise3x3_vec_kernel<ST, 8, VI, HM><<<(unsigned)blocks, 128, 0, stream>>>(x, w, bias, y, g, strips, bands, planes, units)
                if (vin == 4) { if (g.stride == 1) MNNB_DWS_LAUNCH(1, 4, 8); else MNNB_DWS_LAUNCH(2, 4, 8); }
                else if (g.H <= 8) { if (g.stride == 1) MNNB_DWS_LAUNCH(1, 2, 8); else MNNB_DWS_LAUNCH(2, 2, 8); }
                else { if (g.stride == 1) MNNB_DWS_LAUNCH(1, 2, 16); else MNNB_DWS_LAUNCH(2, 2, 16); }
#undef MNNB_DWS_LAUNCH
                return cudaGetLastError();
            }
#define MNNB_DWV_LAUNCH(ST, SWV, VI) depthwise3x3_vec_kernel<ST, SWV, VI><<<(unsigned)blocks, 128, 0, stream>>>(x, w, bias, y, g, strips, bands, planes, units)
#define MNNB_DWV_PICK(ST, VI) do { if (sw == 8) MNNB_DWV_LAUNCH(ST, 8, VI); else if (sw == 16) MNNB_DWV_LAUNCH(ST, 16, VI); else MNNB_DWV_LAUNCH(ST, 32, VI); } while (0)
            if (g.stride == 1) {
                if (vin == 4) MNNB_DWV_PICK(1, 4); else MNNB_DWV_PICK(1, 2);
            } else {
                if (vin == 4) MNNB_DWV_PICK(2, 4); else MNNB_DWV_PICK(2, 2);
            }
#undef MNNB_DWV_PICK
#undef MNNB_DWV_LAUNCH
            return cudaGetLastError();
        }
        // odd widths: one column per lane.  A stride-1 segment of SW lanes covers SW - 1 input columns from -1
        // on, a stride-2 segment SW output columns
        const int need = g.stride == 1 ? g.W + 1 : g.OW;
        const int sw = need <= 8 ? 8 : (need <= 16 ? 16 : 32);
        const int strips = sw < 32 ? 1 : (g.stride == 1 ? (g.OW + 29) / 30 : (g.OW + 31) / 32);
        const long long groups = (planes + 32 / sw - 1) / (32 / sw);
        const long long units = groups * strips * bands;
        const long long blocks = (units + 3) / 4;
        if (blocks > 2147483647ll) return cudaErrorInvalidValue;
#define MNNB_DW_LAUNCH(ST, SWV) depthwise3x3_kernel<ST, SWV><<<(unsigned)blocks, 128, 0, stream>>>(x, w, bias, y, g, strips, bands, planes, units)
        if (g.stride == 1) {
            if (sw == 8) MNNB_DW_LAUNCH(1, 8);
            else if (sw == 16) MNNB_DW_LAUNCH(1, 16);
            else MNNB_DW_LAUNCH(1, 32);
        } else {
            if (sw == 8) MNNB_DW_LAUNCH(2, 8);
            else if (sw == 16) MNNB_DW_LAUNCH(2, 16);
            else MNNB_DW_LAUNCH(2, 32);
        }
#undef MNNB_DW_LAUNCH
        return cudaGetLastError();
    }
    if (direct_stem_applies(g)) {
        const int co_pad = (g.Cout + kStemCoChunk - 1) / kStemCoChunk * kStemCoChunk;
        const size_t smem = (size_t)g.Cin * g.k * g.k * co_pad * sizeof(float);
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(direct_stem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        if (g.Cin == 3 && g.k == 3 && g.dil == 1 && g.stride == 2 && g.pad == 1 && g.H % 2 == 0 && g.W % 4 == 0 &&
            smem <= 48 * 1024 && reinterpret_cast<uintptr_t>(x) % 8 == 0 && reinterpret_cast<uintptr_t>(y) % 8 == 0) {
            const int rows = g.H % 4 == 0 ? 2 : 1;
            const int per_image = (g.OH / rows) * (g.OW / 2);
            const int groups = (per_image + kStemThreads - 1) / kStemThreads;
            const long long units = (long long)g.N * groups;
            if (units <= 2147483647ll) {
                const int resident = 148 * (rows == 1 ? 5 : 3);
                const unsigned blocks = (unsigned)(units < resident ? units : resident);
#define MNNB_STEM_PAIR(RELU, ROWS) direct_stem_s2_pair_kernel<RELU, ROWS><<<blocks, kStemThreads, smem, stream>>>(x, w, bias, y, g, co_pad, groups, (int)units)
                if (rows == 2) { if (g.relu) MNNB_STEM_PAIR(true, 2); else MNNB_STEM_PAIR(false, 2); }
                else { if (g.relu) MNNB_STEM_PAIR(true, 1); else MNNB_STEM_PAIR(false, 1); }
#undef MNNB_STEM_PAIR
                return cudaGetLastError();
            }
        }
        if (g.Cin == 3 && g.k == 3 && g.dil == 1 && (g.stride == 1 || g.stride == 2) && smem <= 48 * 1024) {
            constexpr int kPix = 2;
            const dim3 grid2((unsigned)((g.OH * g.OW + kStemThreads * kPix - 1) / (kStemThreads * kPix)), (unsigned)g.N);
            if (g.stride == 2) direct_stem_fixed_kernel<3, 3, 2, kPix><<<grid2, kStemThreads, smem, stream>>>(x, w, bias, y, g, co_pad);
            else direct_stem_fixed_kernel<3, 3, 1, kPix><<<grid2, kStemThreads, smem, stream>>>(x, w, bias, y, g, co_pad);
            return cudaGetLastError();
        }
        const dim3 grid((unsigned)((g.OH * g.OW + kStemThreads - 1) / kStemThreads), (unsigned)g.N);
        direct_stem_kernel<<<grid, kStemThreads, smem, stream>>>(x, w, bias, y, g, co_pad);
        return cudaGetLastError();
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148ll * 64) blocks = 148ll * 64;
    direct_generic_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, w, bias, y, g, total);
    return cudaGetLastError();
}

}  // namespace mnnb
