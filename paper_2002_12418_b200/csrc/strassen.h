// One recursion level of Strassen's algorithm on the matrix product of a 1x1 convolution (Section 3.3.2, Eq. 9):
// seven half-size products instead of eight, with the additions folded into one pass before and one pass after
// the tensor-core contraction.  Interface between the plan object and strassen.cu.
#pragma once
#include <cuda_runtime.h>

#include "kernels.h"

namespace mnnb {

// y[n][co][p] = act(sum_c w[co][c] x[n][c][p] + bias[co]): C = W X with W [Cout x Cin] and X [Cin x N*HW], split
// into quadrants by halves of Cout, of Cin and of the batch (N even: images [0, N/2) and [N/2, N)).
struct StrassenGeom {
    int N, Cin, Cout, HW;
    int k_pad;                // row length of the half-size operands (Cin / 2 rounded up to 8)
    long long t_half;         // (N / 2) * HW: columns of a half-size product
    long long m_row_stride;   // elements between consecutive output channels of M
};

inline bool strassen_applies(int N, int Cin, int Cout, int k, int stride, int pad, int dil, int groups)
{
    return k == 1 && stride == 1 && pad == 0 && dil == 1 && groups == 1 && N % 2 == 0 && Cout % 2 == 0 && Cin % 2 == 0;
}

// U[xi][co'][c'] (xi < 7, mode = operand format of kernels.h): the seven left operands from the quadrants of w.
cudaError_t launch_strassen_weights(const float* w, void* U_hi, void* U_lo, const StrassenGeom& g, int mode, cudaStream_t stream);
// V[xi][t'][c']: the seven right operands from the quadrants of x, K-major.
cudaError_t launch_strassen_input(const float* x, void* V_hi, void* V_lo, const StrassenGeom& g, int mode, cudaStream_t stream);
// y from the seven products M[xi][co'][t'] (fp32), with bias and ReLU.
cudaError_t launch_strassen_output(const float* M, const float* bias, float* y, const StrassenGeom& g, int relu,
                                   cudaStream_t stream);

}  // namespace mnnb
