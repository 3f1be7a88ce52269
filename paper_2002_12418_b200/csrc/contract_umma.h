// The tcgen05 batched contraction (Section 3.3.1 (2)): interface between the plan object and contract_umma.cu.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "kernels.h"

namespace mnnb {

// tcgen05 contraction.  The object owns the TMA tensor maps of one plan.
struct UmmaContract {
    CUtensorMap map_v_hi, map_v_lo, map_u_hi, map_u_lo;
    int kind;          // 0 tf32, 1 bf16
    int passes;        // 1 or 3
    int alpha2, Cout, cin_pad;
    long long tiles_capacity;
    int bn;            // MMA N (output channels per work item), multiple of 16, <= 256
    int n_co_blocks;
    int k_blocks;
    int stages;
    int stages_sw = 128;               // bytes of K per shared-memory row of a stage (128, or 64 for deeper pipelines)
    int tmem_cols;
    int smem_bytes;
    int num_sms;
    bool a_mn = false;                 // operand A is x itself (1x1 stride-1 convolution), see umma_contract_setup_x
    int x_images = 0, x_cin = 0, x_hw = 0;
    int merged = 0;                    // hi and lo tiles of an operand arrive with one copy (maps with a hi / lo dimension)
    bool ready = false;
};
// Tensor maps over an operand array [planes][rows][k] (k contiguous): box = [1][box_rows][sw bytes of k] with the
// sw-byte swizzle (sw = 128 or 64); and over a hi / lo pair of such arrays (the lo array lo_offset_bytes behind the hi
// array): box = [1][2][box_rows][sw bytes], the hi tile landing first, the lo tile right behind it.
bool encode_operand_map_sw(CUtensorMap* map, void* base, int elem_bytes, long long k_len, long long rows, long long planes,
                           long long plane_stride_elems, int box_rows, int sw);
bool encode_operand_pair_map(CUtensorMap* map, void* base_hi, long long lo_offset_bytes, int elem_bytes, long long k_len,
                             long long rows, long long planes, long long plane_stride_elems, int box_rows, int sw);

// Encodes the tensor maps for U/V at the given device addresses.  Returns a CUDA error or cudaSuccess;
// *why gets a static reason on failure.
cudaError_t umma_contract_setup(UmmaContract* uc, int mode, int alpha2, int Cout, int cin_pad, long long tiles_capacity,
                                void* U_hi, void* U_lo, void* V_hi, void* V_lo, const char** why);
cudaError_t launch_contract_umma(const UmmaContract& uc, long long tiles, const ContractEpilogue& epi, int* status,
                                 cudaStream_t stream);
// 1x1 stride-1 unpadded convolution without a patch matrix: operand A is x [images][Cin][hw] (hw >= 32, a
// multiple of 4, x 16-byte aligned), operand B is U [Cout][cin_pad] in TF32; epi.mode must be 1.
cudaError_t umma_contract_setup_x(UmmaContract* uc, int Cout, int Cin, int cin_pad, int images, int hw, void* U,
                                  const char** why);
cudaError_t launch_contract_umma_x(const UmmaContract& uc, const float* x, const ContractEpilogue& epi, int* status,
                                   cudaStream_t stream);

// 3-D tensor map over an operand tensor [planes][rows][k] (k contiguous), box = [1][box_rows][128 bytes of k],
// 128-byte swizzle; elements outside the tensor read as zero.  False when the driver entry point is missing
// or refuses the shape.
bool encode_operand_map(CUtensorMap* map, void* base, int elem_bytes, long long k_len, long long rows, long long planes,
                        long long plane_stride_elems, int box_rows);

// One thread waits, with the bounded wait of umma.cuh, on a barrier nobody arrives on; *device_word ends as 2.
cudaError_t launch_wait_probe(int* device_word, cudaStream_t stream);

}  // namespace mnnb
