// Implicit GEMM for convolutions with k > 1 and stride / dilation / padding (the GEMM scheme without a patch
// matrix): y[n][co][oh][ow] = act(sum_kk U[co][kk] patch(n, oh, ow)[kk] + bias[co]), kk = (ci * k + a) * k + b,
// where the patches are gathered by producer warps straight into the shared-memory operand tile of the tensor
// core and never stored.  Interface between the plan object and implicit_gemm.cu.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "kernels.h"

namespace mnnb {

struct ImplicitGemm {
    CUtensorMap map_u;      // U [Cout][k_pad] TF32-rounded fp32 (the GEMM scheme's weight copy), box = bn x 32
    int Cout = 0, k_pad = 0, bn = 0, n_co_blocks = 0, k_blocks = 0, stages = 0, tmem_cols = 0, smem_bytes = 0, num_sms = 0;
    bool ready = false;
};

// The weight copy this kernel reads: U [Cout][k_pad] TF32-rounded, patch elements in the order (ci, a, b) of w, or
// (a, b, ci) when Cin is a multiple of 32 (then a pipeline stage is 32 channels of one kernel tap, which the
// producers gather with one bounds test and loads one channel plane apart).
bool implicit_gemm_tap_major(int Cin);
cudaError_t launch_implicit_weights(const float* w, void* U, int Cout, int Cin, int k, int k_pad, cudaStream_t stream);

// g.k_pad = row length of U (Cin * k * k rounded up to 8).  U must be 16-byte aligned.
cudaError_t implicit_gemm_setup(ImplicitGemm* ig, const GatherGeom& g, int Cout, void* U, const char** why);
cudaError_t launch_implicit_gemm(const ImplicitGemm& ig, const float* x, const float* bias, float* y, const GatherGeom& g,
                                 int relu, int* status, cudaStream_t stream);

}  // namespace mnnb
