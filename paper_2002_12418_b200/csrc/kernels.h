// Internal interface between the plan object and the CUDA kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace mnnb {

// Launch with programmatic stream serialisation allowed: the kernel may be scheduled while the previous
// kernel of the stream is still finishing, provided that kernel has triggered its dependents.  Every kernel
// launched this way calls grid_dependency_wait() (umma.cuh) before it touches global memory, which blocks
// until the previous kernel has completed and its writes are visible; so only launch latency and the
// kernel's own set-up overlap.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// How transformed operands are stored.
enum StoreMode {
    STORE_TF32 = 0,       // fp32 container, rounded to 10 mantissa bits
    STORE_BF16 = 1,       // bf16
    STORE_TF32_SPLIT = 2, // hi and lo, both TF32-rounded fp32
    STORE_BF16_SPLIT = 3, // hi and lo, both bf16
    STORE_FP32 = 4        // unrounded fp32 (checking path)
};

inline int store_elem_bytes(int mode) { return (mode == STORE_BF16 || mode == STORE_BF16_SPLIT) ? 2 : 4; }
inline bool store_is_split(int mode) { return mode == STORE_TF32_SPLIT || mode == STORE_BF16_SPLIT; }

struct TransformMatrices {
    float At[6 * 12];     // [m][alpha]
    float G[12 * 7];      // [alpha][k]
    float Bt[12 * 12];    // [alpha][alpha]
};

// Geometry of one Winograd chunk launch.
struct WinoGeom {
    int images;           // images in this chunk
    int Cin, Cout, H, W, OH, OW, k, pad, m, alpha;
    int th, tw;           // tiles per image, vertically and horizontally
    int cin_pad;          // row length of U and V in elements
    long long tiles;      // images * th * tw
    long long v_plane;    // elements between consecutive transform positions of V (>= tiles * cin_pad)
    long long m_row_stride;   // elements between consecutive output channels of M
};

// U = G w G^T (Eq. 6).  U_hi/U_lo: [alpha^2][Cout][cin_pad] in `mode` format.
cudaError_t launch_weight_transform(const float* w, void* U_hi, void* U_lo, int Cout, int Cin, int k, int m, int cin_pad,
                                    int mode, const TransformMatrices& mats, cudaStream_t stream);
// GEMM scheme: rounded copy of w [Cout][Cin*k*k] into U [Cout][k_pad].
cudaError_t launch_weight_round(const float* w, void* U_hi, void* U_lo, int Cout, int Kd, int k_pad, int mode,
                                cudaStream_t stream);
// V = B^T d B for every tile of the chunk.  x points at the chunk's first image.  `status` (device, may be
// NULL) receives a code if a bounded wait inside the kernel runs out.
cudaError_t launch_input_transform(const float* x, void* V_hi, void* V_lo, const WinoGeom& g, int mode,
                                   const TransformMatrices& mats, int* status, cudaStream_t stream);
// y = act(A^T M A + bias).  y points at the chunk's first image.
cudaError_t launch_output_transform(const float* M, const float* bias, float* y, const WinoGeom& g, int relu,
                                    const TransformMatrices& mats, cudaStream_t stream);

// Patch gather for the GEMM scheme: V[t][(ci*k + a)*k + b] = xpad[...], t = (n*OH + oh)*OW + ow.
struct GatherGeom {
    int N, Cin, H, W, OH, OW, k, stride, pad, dil, k_pad;
};
cudaError_t launch_gather(const float* x, void* V_hi, void* V_lo, const GatherGeom& g, int mode, cudaStream_t stream);

// Epilogue of a contraction: 0 = write M[xi][co][t]; 1 = write y[n][co][pix] = act(. + bias), t = n*ohw + pix.
struct ContractEpilogue {
    int mode;
    float* M;
    long long m_row_stride;
    float* y;
    const float* bias;
    int relu;
    int ohw;
};

// CUDA-core fp32 contraction (checking path): out[xi][co][t] = sum_c U[xi][co][c] * V[xi][t][c].
cudaError_t launch_contract_reference(const void* U_hi, const void* U_lo, const void* V_hi, const void* V_lo, int mode,
                                      int alpha2, int Cout, long long tiles, int cin_pad, long long u_plane,
                                      long long v_plane, const ContractEpilogue& epi, cudaStream_t stream);

// Direct ("sliding window") convolution, any stride / padding / dilation / groups.
struct DirectGeom {
    int N, Cin, Cout, H, W, OH, OW, k, stride, pad, dil, groups, relu;
};
cudaError_t launch_direct(const float* x, const float* w, const float* bias, float* y, const DirectGeom& g,
                          cudaStream_t stream);
// True when the direct path uses its kernel for layers with very few input channels (Cin <= 4, groups 1).
bool direct_stem_applies(const DirectGeom& g);

}  // namespace mnnb
