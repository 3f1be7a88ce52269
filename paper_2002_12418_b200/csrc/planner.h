// Pre-inference planner: scheme selection by an integer cost model (Eq. 1-5
// re-stated for one B200) with an accuracy gate.  Host only.
#pragma once
#include <cstdint>

#include "../../include/mnn_conv.h"

namespace mnnb {

struct LayerShape {
    int N, Cin, Cout, H, W, k, stride, pad, dil, groups, relu;
    int OH, OW;
};

struct Calibration {
    long long c[MNN_N_CONSTS];
};

struct Decision {
    int algo = 0, m = 0, alpha = 0, operand = 0, passes = 0, points_id = 0;
    int chunk_images = 0, n_chunks = 0;
    int chosen = -1;
    int gemm_lhs = 0;                  // MNN_GEMM_LHS_PATCHES or MNN_GEMM_LHS_X for the GEMM scheme, else 0
    int fused = 0;                     // Winograd F(2x2,3x3) as the single fused kernel
    int paper_n_hat = 0;               // Eq. 2's argmin over n in {1, 2, 4, 6} and the counts themselves
    uint64_t paper_mul[4] = {0, 0, 0, 0};
    long long error_ppm = 0;
    uint64_t cost_ps[MNN_N_CANDIDATES];
};

// Relative L2 error x 1e6 of the GEMM scheme when the tensor core truncates x to TF32 itself (measured; it is a
// bias toward zero, so it does not grow with the length of the sums).
constexpr long long kGemmLhsXErrorPpm = 340;

constexpr int kGateNumerator = 7;      // admissible when predicted error <= 0.7 x the class tolerance
constexpr int kGateDenominator = 10;

Calibration default_calibration();
Calibration current_calibration();
void install_calibration(const Calibration& c);

// Output channels per work item (MMA N) of the tensor-core contraction and the number of channel blocks, for
// `tile_blocks` blocks of 128 tiles per transform position: a multiple of 16, at most 256, blocks balanced.
// Wider blocks re-use the tile operand more, narrower ones give more work items; among 1x, 2x and 4x the
// minimum number of blocks the shortest schedule wins: rounds of work items over the SMs times the operand
// rows an item loads (128 tiles + bn channels).  The kernel's host side and the cost model both call this.
void contract_tiling(long long tile_blocks, int alpha2, int Cout, int num_sms, int* bn, int* n_co_blocks);

// True when the GEMM scheme can take x itself as its left operand (no patch matrix): a 1x1 stride-1 unpadded
// ungrouped layer with H*W >= 32 and a multiple of 4, single-pass TF32 operands.
bool gemm_reads_x(const LayerShape& s, int operand, int passes);

// Output extent of one spatial dimension; 0 when the kernel does not fit.
int conv_out_extent(int in, int k, int stride, int pad, int dil);

// Predicted relative L2 error x 1e6 (deterministic host simulation).  m = 1 and
// points_id = 0 gives the GEMM figure.  -1 on invalid arguments.
long long accuracy_ppm(int m, int k, int points_id, int operand, int passes);

// Best point set for (m, k, operand, passes): lowest predicted error, ties to the lower id.
int best_points(int m, int k, int operand, int passes, long long* ppm_out);

// Images per chunk and whether the chunk's V and M stay L2-resident, for a Winograd candidate.
void winograd_chunking(const LayerShape& s, int m, int operand, int passes, const Calibration& cal,
                       int* chunk_images, int* n_chunks, uint64_t* cost_ps);

// Fills *d.  Returns MNN_OK or an mnn_status with *err set to a static reason.
// True when the layer's shape admits the fused Winograd F(2x2, 3x3) kernel.
bool fused_shape_ok(const LayerShape& s);

int plan_layer(const LayerShape& s, const mnn_conv_opts& o, const Calibration& cal, Decision* d, const char** err);

// True when the Winograd kernels exist for (m, k).
bool winograd_supported(int m, int k);

}  // namespace mnnb
