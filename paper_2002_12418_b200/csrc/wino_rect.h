// Rectangular kernels (1 x k and k x 1; the paper's Section 4.2 names Inception-v3's 1 x 7 / 7 x 1 layers):
// Winograd along the long axis only, F(m, k) in one dimension (Eq. 6 with the identity on the other axis):
//     y = A^T [ sum_c (G w) (.) (B^T d) ]
// with alpha = m + k - 1 transform positions.  Interface between the plan object and wino_rect.cu.
#pragma once
#include <cuda_runtime.h>

#include "kernels.h"

namespace mnnb {

struct RectGeom {
    int N, Cin, Cout, H, W, OH, OW;
    int k;              // length of the kernel along its long axis
    int along_w;        // 1: kernel 1 x k (tiles along the width), 0: kernel k x 1 (tiles along the height)
    int pad_h, pad_w;
    int m, alpha;
    int n_seg;          // tiles per output line: ceil(OW / m) or ceil(OH / m)
    int cin_pad;
    long long tiles;    // along_w: N * OH * n_seg (t = (n * OH + oh) * n_seg + seg); else N * n_seg * OW (t = (n * n_seg + seg) * OW + ow)
    long long m_row_stride;
};

constexpr int kRectMaxAlpha = 10;

// U[xi][co][ci] = sum_a G[xi][a] w[co][ci][a]   (w is [Cout][Cin][k], the kernel's long axis contiguous)
cudaError_t launch_rect_weights(const float* w, void* U_hi, void* U_lo, const RectGeom& g, int mode, const TransformMatrices& mats,
                                cudaStream_t stream);
// V[xi][t][ci] = sum_j Bt[xi][j] xpad[n][ci][line position of tile t + j]
cudaError_t launch_rect_input(const float* x, void* V_hi, void* V_lo, const RectGeom& g, int mode, const TransformMatrices& mats,
                              cudaStream_t stream);
// y = act(A^T M + bias) from M[xi][co][t] (fp32)
cudaError_t launch_rect_output(const float* M, const float* bias, float* y, const RectGeom& g, int relu, const TransformMatrices& mats,
                               cudaStream_t stream);

}  // namespace mnnb
