// The Winograd contraction on pairs of SMs (contract_pair.cu): interface between the plan object and the kernel.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace mnnb {

struct PairContract {
    CUtensorMap map_v_hi, map_v_lo, map_u_hi, map_u_lo;
    int kind = 0;          // 0 tf32, 1 bf16
    int passes = 1;        // 1 or 3 (hi + lo operands)
    int alpha2 = 0, Cout = 0, cin_pad = 0;
    long long tiles_capacity = 0;
    int bn = 256;          // output channels per work item (MMA N, a multiple of 32, at most 256)
    int k_blocks = 0, stages = 0, sw = 128, merged = 0, num_sms = 0, smem_bytes = 0;
    bool ready = false;
};

// True when the pair kernel applies: a Winograd contraction (alpha2 > 1) over TF32 or BF16 operands whose
// device has an even number of SMs.  *why gets a static reason otherwise.
cudaError_t pair_contract_setup(PairContract* pc, int mode, int alpha2, int Cout, int cin_pad, long long tiles_capacity, void* U_hi,
                                void* U_lo, void* V_hi, void* V_lo, const char** why);
// out = M [alpha2][Cout][m_row_stride], tiles <= tiles_capacity rows of V per position.
cudaError_t launch_contract_pair(const PairContract& pc, long long tiles, float* M, long long m_row_stride, int* status,
                                 cudaStream_t stream);

}  // namespace mnnb
