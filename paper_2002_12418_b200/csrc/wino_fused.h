// Winograd F(2x2, 3x3) in one kernel: input transform, tensor-core contraction and output transform fused, so
// that the transformed tensors V and M never reach global memory (Eq. 6).  Interface between the plan object
// and wino_fused.cu.
#pragma once
#include <cuda_runtime.h>

#include "kernels.h"

namespace mnnb {

// The transformed weights U = G w G^T are stored PACKED for this kernel: in the byte order the tensor core
// reads them from shared memory, so that a block of them is one contiguous bulk copy.
//   U_packed [channel block of 128 outputs][block of 16 input channels][16 transform positions][128 rows][64 bytes]
// where a row holds the 16 input channels of one output channel in TF32 (fp32 container) with the four
// 16-byte pieces of the row permuted by (row / 2) mod 4 (the 64-byte swizzle of the shared-memory operand
// layout); rows beyond Cout and channels beyond Cin hold zeros.
long long fused_wino_weight_bytes(int Cout, int Cin);

struct FusedWino {
    const void* U = nullptr;
    int Cout = 0, Cin = 0, num_sms = 0, smem_bytes = 0;
    bool ready = false;
};

// True when the layer's shape admits this kernel.
bool fused_wino_applies(int k, int stride, int dil, int groups, int pad, long long tiles);
cudaError_t fused_wino_setup(FusedWino* fw, int Cout, int Cin, const void* U_packed, const char** why);
// U_packed = packed G w G^T of w [Cout][Cin][3][3], rounded to TF32 (preparation time).
cudaError_t launch_fused_wino_weights(const float* w, void* U_packed, int Cout, int Cin, const TransformMatrices& mats,
                                      cudaStream_t stream);
// y = act(A^T [ sum_c U (.) (B^T x B) ] A + bias) for the whole batch in one launch.
cudaError_t launch_fused_wino(const FusedWino& fw, const float* x, const float* bias, float* y, const WinoGeom& g, int relu,
                              const TransformMatrices& mats, int* status, cudaStream_t stream);

}  // namespace mnnb
