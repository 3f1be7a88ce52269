// Templates of the Winograd input and output transform kernels; instantiated per
// alpha in wino_inst_*.cu so that the translation units compile in parallel.
#pragma once
#include <cuda_bf16.h>

#include "kernels.h"
#include "wino_input.cuh"

namespace mnnb {
namespace wino {

struct MatBt { float v[12 * 12]; };
struct MatAt { float v[6 * 12]; };
struct MatG { float v[12 * 7]; };

__device__ __forceinline__ float round_tf32(float v)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

// Store one transformed value in the operand format(s).
__device__ __forceinline__ void store_operand(void* hi, void* lo, size_t idx, float v, int mode)
{
    switch (mode) {
        case STORE_TF32:
            reinterpret_cast<float*>(hi)[idx] = round_tf32(v);
            break;
        case STORE_BF16:
            reinterpret_cast<__nv_bfloat16*>(hi)[idx] = __float2bfloat16_rn(v);
            break;
        case STORE_TF32_SPLIT: {
            const float h = round_tf32(v);
            reinterpret_cast<float*>(hi)[idx] = h;
            reinterpret_cast<float*>(lo)[idx] = round_tf32(v - h);
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

// ---------------------------------------------------------------------------
// Output transform: one thread per (tile, output channel); consecutive threads
// take consecutive tiles, so the alpha^2 reads of M[xi][co][tile] are coalesced
// and the m-wide row pieces written to y are adjacent in memory.
// ---------------------------------------------------------------------------
constexpr int kOutThreads = 128;

template <int ALPHA, int M>
__global__ void __launch_bounds__(kOutThreads) output_transform_kernel(const float* __restrict__ Mx,
                                                                       const float* __restrict__ bias,
                                                                       float* __restrict__ y, WinoGeom g, int relu, MatAt At)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const long long tile = (long long)blockIdx.x * kOutThreads + threadIdx.x;
    const int co = blockIdx.y;
    if (tile >= g.tiles) return;
    float acc[ALPHA][ALPHA];
    const float* src = Mx + (size_t)co * g.m_row_stride + tile;
    const size_t plane = (size_t)g.Cout * g.m_row_stride;
#pragma unroll
    for (int i = 0; i < ALPHA; ++i)
#pragma unroll
        for (int j = 0; j < ALPHA; ++j) acc[i][j] = __ldcs(src + (size_t)(i * ALPHA + j) * plane);

    float t[M][ALPHA];
#pragma unroll
    for (int a = 0; a < M; ++a)
#pragma unroll
        for (int j = 0; j < ALPHA; ++j) {
            float s = 0.0f;
#pragma unroll
            for (int i = 0; i < ALPHA; ++i) s = fmaf(At.v[a * ALPHA + i], acc[i][j], s);
            t[a][j] = s;
        }
    const int tx = (int)(tile % g.tw);
    const long long rest = tile / g.tw;
    const int ty = (int)(rest % g.th);
    const int img = (int)(rest / g.th);
    const float b = bias ? __ldg(bias + co) : 0.0f;
    float* dst = y + (((size_t)img * g.Cout + co) * g.OH + (size_t)ty * M) * g.OW + (size_t)tx * M;
    const int rows = min(M, g.OH - ty * M), cols = min(M, g.OW - tx * M);
#pragma unroll
    for (int a = 0; a < M; ++a) {
        float o[M];
#pragma unroll
        for (int c = 0; c < M; ++c) {
            float s = b;
#pragma unroll
            for (int j = 0; j < ALPHA; ++j) s = fmaf(t[a][j], At.v[c * ALPHA + j], s);
            o[c] = relu ? fmaxf(s, 0.0f) : s;
        }
        if (a < rows) {
            float* row = dst + (size_t)a * g.OW;
            if (cols == M && (M % 2 == 0) && ((reinterpret_cast<uintptr_t>(row) & 7u) == 0)) {
#pragma unroll
                for (int c = 0; c < M; c += 2) *reinterpret_cast<float2*>(row + c) = make_float2(o[c], o[c + 1]);
            } else {
#pragma unroll
                for (int c = 0; c < M; ++c)
                    if (c < cols) row[c] = o[c];
            }
        }
    }
}

template <int ALPHA, int M>
cudaError_t launch_output_am(const float* Mx, const float* bias, float* y, const WinoGeom& g, int relu,
                             const TransformMatrices& mats, cudaStream_t stream)
{
    MatAt at;
    for (int i = 0; i < M * ALPHA; ++i) at.v[i] = mats.At[i];
    dim3 grid((unsigned)((g.tiles + kOutThreads - 1) / kOutThreads), (unsigned)g.Cout);
    return launch_overlapped(output_transform_kernel<ALPHA, M>, grid, dim3(kOutThreads), 0, stream, Mx, bias, y, g, relu, at);
}


}  // namespace wino
}  // namespace mnnb

// One non-template entry point per instantiation, defined in wino_inst_*.cu.
#define MNNB_INPUT_FN(A) launch_input_transform_a##A
#define MNNB_OUTPUT_FN(A, MM) launch_output_transform_a##A##_m##MM
#define MNNB_INPUT_ARGS const float *x, void *V_hi, void *V_lo, const WinoGeom &g, int mode, const TransformMatrices &mats, int *status, int num_sms, cudaStream_t stream
#define MNNB_OUTPUT_ARGS const float *Mx, const float *bias, float *y, const WinoGeom &g, int relu, const TransformMatrices &mats, cudaStream_t stream
#define MNNB_DEFINE_INPUT(A) \
    namespace mnnb { cudaError_t MNNB_INPUT_FN(A)(MNNB_INPUT_ARGS) { return wino::launch_input_ws<A>(x, V_hi, V_lo, g, mode, mats, status, num_sms, stream); } }
#define MNNB_DEFINE_OUTPUT(A, MM) \
    namespace mnnb { cudaError_t MNNB_OUTPUT_FN(A, MM)(MNNB_OUTPUT_ARGS) { return wino::launch_output_am<A, MM>(Mx, bias, y, g, relu, mats, stream); } }
#define MNNB_DECLARE_INPUT(A) namespace mnnb { cudaError_t MNNB_INPUT_FN(A)(MNNB_INPUT_ARGS); }
#define MNNB_DECLARE_OUTPUT(A, MM) namespace mnnb { cudaError_t MNNB_OUTPUT_FN(A, MM)(MNNB_OUTPUT_ARGS); }
