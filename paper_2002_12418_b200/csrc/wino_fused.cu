// Winograd F(2x2, 3x3) as ONE kernel (Eq. 6): y = A^T [ sum_c (G w G^T) (.) (B^T d B) ] A + bias, ReLU.
//
// The three stages of Eq. 6 run inside one persistent CTA per SM, so that neither the transformed input V
// nor the products M ever reach HBM (Section 3.3.1 (2) notes that memory access dominates the Hadamard form;
// this removes the two largest tensors from memory altogether):
//   - eight producer warps read the 4 x 4 input windows of a block of 32 tiles, compute B^T d B in registers
//     (packed fp32 pairs, two channels per lane) and write the sixteen transform positions, rounded to TF32,
//     straight into shared memory in the 128-byte-swizzled K-major layout the tensor core reads;
//   - one thread streams the transformed weights U[xi][co][ci] (prepared once, Eq. 6's G w G^T) with TMA,
//     one 128 x 32 box per transform position and block of 32 input channels, through a ring of stages;
//   - one thread issues tcgen05.mma (kind::tf32, M = 128 output channels, N = 32 tiles, K = 8 per instruction)
//     into SIXTEEN accumulators, one per transform position, which together fill the 512 columns of tensor
//     memory;
//   - four epilogue warps read the sixteen accumulators of their output channels with tcgen05.ld, apply
//     A^T . A, bias and ReLU in registers, transpose through a small staging buffer so that consecutive lanes
//     hold consecutive tiles, and store rows of y.
// A work item is (block of 32 consecutive tiles, block of 128 output channels).  Tensor memory holds exactly
// one item, so the epilogue of an item and the MMAs of the next do not overlap; the producers and the weight
// stream run ahead meanwhile.  Every mbarrier wait is bounded and reports through the status word.
#include <cstring>

#include "kernels.h"
#include "umma.cuh"
#include "wino_input.cuh"

namespace mnnb {

namespace {

constexpr int kProducerWarps = 8;
constexpr int kEpilogueWarps = 4;
constexpr int kThreads = 32 * (2 + kEpilogueWarps + kProducerWarps);   // warp 0 TMA, warp 1 MMA, epilogue, producers
constexpr int kTiles = 32;             // tiles per work item (MMA N)
constexpr int kCo = 128;               // output channels per work item (MMA M)
constexpr int kKBlock = 32;            // input channels per pipeline step: one 128-byte row of TF32
constexpr int kPositions = 16;         // alpha^2
constexpr int kUStageBytes = kCo * 128;                    // one transform position of U for one K block
constexpr int kVBytes = kPositions * kTiles * 128;         // all positions of V for one K block
constexpr int kStageRow = 8 * 4 + 4;                       // staging: 8 tiles x 4 outputs per channel, + 4 words of padding
constexpr int kStagingBytes = kEpilogueWarps * 32 * kStageRow * 4;
constexpr int kMaxUStages = 9;
constexpr int kSmemBudget = 226 * 1024;

constexpr int kErrTmaWait = 21, kErrMmaWaitU = 22, kErrMmaWaitV = 23, kErrMmaWaitAcc = 24, kErrEpilogueWait = 25,
              kErrProducerWait = 26;

struct MatAt4 { float v[2 * 4]; };     // A^T of F(2, 3): [2][4]

struct FusedParams {
    const float* x;
    const float* bias;
    float* y;
    int images, Cin, Cout, H, W, OH, OW, pad, th, tw, relu;
    int tiles;               // images * th * tw
    int n_tile_blocks, n_co_blocks, k_blocks, u_stages;
    int n_items;
    int sym;                 // B^T has the symmetric-point structure
    int* status;
};

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&r)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ float2 tf32_pair(float2 v)
{
    return make_float2(wino::round_tf32_v(v.x), wino::round_tf32_v(v.y));
}

__global__ void __launch_bounds__(kThreads, 1)
fused_f2x2_3x3_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ wino::MatBt2 Bt, MatAt4 At,
                      FusedParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t u_full[kMaxUStages];
    __shared__ __align__(8) uint64_t u_empty[kMaxUStages];
    __shared__ __align__(8) uint64_t v_full, v_empty, acc_full, acc_empty;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    volatile int* abortp = &abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t v_base = smem_base;                                 // V: [position][tile][32 channels], swizzled
    const uint32_t u_base = smem_base + kVBytes;                       // U ring
    uint8_t* const generic_base = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    float* const staging = reinterpret_cast<float*>(generic_base + kVBytes + p.u_stages * kUStageBytes);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.u_stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&u_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&u_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&v_full), kProducerWarps);
        ptx::mbar_init(ptx::smem_u32(&v_empty), 1);
        ptx::mbar_init(ptx::smem_u32(&acc_full), 1);
        ptx::mbar_init(ptx::smem_u32(&acc_empty), kEpilogueWarps);
        abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_u);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512u);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    const int first = blockIdx.x, step = gridDim.x;

    if (warp == 0) {
        // ------------------------------ weight stream (TMA) ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int item = first; item < p.n_items && ok; item += step) {
                const int cb = item / p.n_tile_blocks;
                for (int kb = 0; kb < p.k_blocks && ok; ++kb)
                    for (int xi = 0; xi < kPositions; ++xi) {
                        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&u_empty[stage]), phase ^ 1u, abortp)) {
                            if (!*abortp) atomicCAS(p.status, 0, kErrTmaWait);
                            *abortp = 1;
                            ok = false;
                            break;
                        }
                        const uint32_t bar = ptx::smem_u32(&u_full[stage]);
                        ptx::mbar_expect_tx(bar, kUStageBytes);
                        ptx::tma_load_3d(u_base + stage * kUStageBytes, &map_u, bar, kb * kKBlock, cb * kCo, xi);
                        if (++stage == (uint32_t)p.u_stages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issue ------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::mma_idesc(2, kCo, kTiles);
            uint32_t stage = 0, phase = 0, v_phase = 0, acc_phase = 0;
            bool ok = true;
            for (int item = first; item < p.n_items && ok; item += step) {
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&acc_empty), acc_phase ^ 1u, abortp)) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitAcc);
                    *abortp = 1;
                    break;
                }
                ptx::tc_fence_after();
                for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&v_full), v_phase, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitV);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    for (int xi = 0; xi < kPositions; ++xi) {
                        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&u_full[stage]), phase, abortp)) {
                            if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitU);
                            *abortp = 1;
                            ok = false;
                            break;
                        }
                        ptx::tc_fence_after();
                        const uint32_t a_addr = u_base + stage * kUStageBytes;
                        const uint32_t b_addr = v_base + (uint32_t)xi * (kTiles * 128);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            ptx::mma_ss<0>(tmem_base + (uint32_t)xi * kTiles, ptx::smem_desc_k128(a_addr + ks * 32),
                                           ptx::smem_desc_k128(b_addr + ks * 32), idesc, (kb | ks) != 0 ? 1u : 0u);
                        ptx::mma_commit(ptx::smem_u32(&u_empty[stage]));
                        if (++stage == (uint32_t)p.u_stages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    ptx::mma_commit(ptx::smem_u32(&v_empty));          // V may be overwritten once these MMAs retire
                    v_phase ^= 1u;
                }
                if (!ok) break;
                ptx::mma_commit(ptx::smem_u32(&acc_full));
                acc_phase ^= 1u;
            }
        }
    } else if (warp < 2 + kEpilogueWarps) {
        // ------------------------------ epilogue: A^T . A, bias, ReLU, store ------------------------------
        const int q = warp & 3;                                      // quarter of the tensor-memory lanes this warp may read
        float* const stg = staging + (warp - 2) * 32 * kStageRow;
        uint32_t acc_phase = 0;
        const bool y_pairs = (p.OW % 2 == 0) && ((reinterpret_cast<uintptr_t>(p.y) & 7u) == 0);
        for (int item = first; item < p.n_items; item += step) {
            const int cb = item / p.n_tile_blocks, tb = item - cb * p.n_tile_blocks;
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_relaxed(ptx::smem_u32(&acc_full), acc_phase, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrEpilogueWait);
                    *abortp = 1;
                }
                break;
            }
            ptx::tc_fence_after();
            const int co_lane = cb * kCo + q * 32 + lane;             // the channel whose accumulators this lane reads
            const float b = (p.bias && co_lane < p.Cout) ? __ldg(p.bias + co_lane) : 0.0f;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            for (int rd = 0; rd < kTiles / 8; ++rd) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t m[kPositions][4];
#pragma unroll
                    for (int xi = 0; xi < kPositions; ++xi) tmem_ld4(taddr + (uint32_t)(xi * kTiles + rd * 8 + half * 4), m[xi]);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        // rows: s[a][j] = sum_i At[a][i] M[i][j]; then o[a][b] = sum_j s[a][j] At[b][j]
                        float s[2][4];
#pragma unroll
                        for (int a = 0; a < 2; ++a)
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                float acc = At.v[a * 4] * __uint_as_float(m[j][t]);
#pragma unroll
                                for (int i = 1; i < 4; ++i) acc = fmaf(At.v[a * 4 + i], __uint_as_float(m[i * 4 + j][t]), acc);
                                s[a][j] = acc;
                            }
                        float o[4];
#pragma unroll
                        for (int a = 0; a < 2; ++a)
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                float acc = b;
#pragma unroll
                                for (int j = 0; j < 4; ++j) acc = fmaf(s[a][j], At.v[c * 4 + j], acc);
                                o[a * 2 + c] = p.relu ? fmaxf(acc, 0.0f) : acc;
                            }
                        *reinterpret_cast<float4*>(stg + lane * kStageRow + (half * 4 + t) * 4) = make_float4(o[0], o[1], o[2], o[3]);
                    }
                }
                __syncwarp();
                // read back with lanes = (tile j, output row r, channel parity): rows of y
                {
                    const int j = lane & 7, r = (lane >> 3) & 1, cs = lane >> 4;
                    const int tile = tb * kTiles + rd * 8 + j;
                    const bool tile_ok = tile < p.tiles;
                    const int tt = tile_ok ? tile : 0;
                    const int tx = tt % p.tw, rest = tt / p.tw;
                    const int ty = rest % p.th, img = rest / p.th;
                    const int oh = ty * 2 + r, ow = tx * 2;
                    const bool row_ok = tile_ok && oh < p.OH;
                    const size_t plane = (size_t)p.OH * p.OW;
                    float* const ybase = p.y + (size_t)img * p.Cout * plane + (size_t)oh * p.OW + ow;
#pragma unroll 4
                    for (int c2 = 0; c2 < 16; ++c2) {
                        const int cl = c2 * 2 + cs;
                        const int co = cb * kCo + q * 32 + cl;
                        const float2 v = *reinterpret_cast<const float2*>(stg + cl * kStageRow + j * 4 + r * 2);
                        if (row_ok && co < p.Cout) {
                            float* dst = ybase + (size_t)co * plane;
                            if (y_pairs) {
                                *reinterpret_cast<float2*>(dst) = v;           // OW even: both columns exist
                            } else {
                                dst[0] = v.x;
                                if (ow + 1 < p.OW) dst[1] = v.y;
                            }
                        }
                    }
                }
                __syncwarp();
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&acc_empty));
            acc_phase ^= 1u;
        }
    } else {
        // ------------------------------ producers: V = B^T d B into shared memory ------------------------------
        // A warp owns 8 consecutive tiles of the block (lane & 7) and, per step, 4 channel pairs (lane >> 3):
        // the 8-byte stores of a half-warp then fall into distinct 16-byte columns of the swizzled rows.
        const int pw = warp - 2 - kEpilogueWarps;
        const int t8 = lane & 7, cp4 = lane >> 3;
        const int tg = pw & 3;                                        // which 8 tiles of the 32
        const int cg0 = pw >> 2;                                      // channel-pair groups cg0 and cg0 + 2 (of 4)
        const int row = tg * 8 + t8;                                  // the tile's row in every V[xi] matrix
        uint32_t v_phase = 0;
        bool ok = true;
        const size_t plane = (size_t)p.H * p.W;
        for (int item = first; item < p.n_items && ok; item += step) {
            const int cb = item / p.n_tile_blocks, tb = item - cb * p.n_tile_blocks;
            (void)cb;
            const int tile = tb * kTiles + row;
            const bool tile_ok = tile < p.tiles;
            const int tt = tile_ok ? tile : 0;
            const int tx = tt % p.tw, rest = tt / p.tw;
            const int ty = rest % p.th, img = rest / p.th;
            const int ih0 = ty * 2 - p.pad, iw0 = tx * 2 - p.pad;
            // which of the 4 x 4 window positions lie inside the image
            unsigned mask = 0;
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (tile_ok && ih0 + r >= 0 && ih0 + r < p.H && iw0 + c >= 0 && iw0 + c < p.W) mask |= 1u << (r * 4 + c);
            const float* const xwin = p.x + (size_t)img * p.Cin * plane + (ptrdiff_t)ih0 * p.W + iw0;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                // both tasks' windows are loaded before the wait, so that the loads overlap it
                float2 d[2][4][4];
#pragma unroll
                for (int task = 0; task < 2; ++task) {
                    const int c = kb * kKBlock + (cg0 + 2 * task) * 8 + cp4 * 2;
                    const float* p0 = xwin + (size_t)c * plane;
                    const bool c0_ok = c < p.Cin, c1_ok = c + 1 < p.Cin;
#pragma unroll
                    for (int r = 0; r < 4; ++r)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            const bool in = (mask >> (r * 4 + cc)) & 1u;
                            const ptrdiff_t off = (ptrdiff_t)r * p.W + cc;
                            d[task][r][cc].x = (in && c0_ok) ? __ldg(p0 + off) : 0.0f;
                            d[task][r][cc].y = (in && c1_ok) ? __ldg(p0 + plane + off) : 0.0f;
                        }
                }
                int got = 1;
                if (lane == 0) got = ptx::mbar_wait_relaxed(ptx::smem_u32(&v_empty), v_phase ^ 1u, abortp) ? 1 : 0;
                got = __shfl_sync(0xffffffffu, got, 0);
                if (!got) {
                    if (lane == 0) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrProducerWait);
                        *abortp = 1;
                    }
                    ok = false;
                    break;
                }
#pragma unroll
                for (int task = 0; task < 2; ++task) {
                    float2 h[4][4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        if (p.sym) wino::pass_1d<4, true, float2>(d[task][r], h[r], Bt);
                        else wino::pass_1d<4, false, float2>(d[task][r], h[r], Bt);
                    }
                    // byte offset of this lane's channel pair inside its (swizzled) row
                    const int chunk = (cg0 + 2 * task) * 2 + (cp4 >> 1);           // 16-byte column 0..7
                    const uint32_t in_row = (uint32_t)(((chunk ^ (row & 7)) << 4) | ((cp4 & 1) << 3));
                    uint8_t* const dst = generic_base + row * 128 + in_row;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float2 col[4], o[4];
#pragma unroll
                        for (int r = 0; r < 4; ++r) col[r] = h[r][j];
                        if (p.sym) wino::pass_1d<4, true, float2>(col, o, Bt);
                        else wino::pass_1d<4, false, float2>(col, o, Bt);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            *reinterpret_cast<float2*>(dst + (i * 4 + j) * (kTiles * 128)) = tf32_pair(o[i]);
                    }
                }
                fence_proxy_async_smem();                      // the tensor core reads these through the async proxy
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&v_full));
                v_phase ^= 1u;
            }
        }
    }

    // Teardown.  After an aborted run give copies still in flight time to land before shared memory is released.
    if (*abortp) __nanosleep(200000);
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512u);
    }
}

}  // namespace

bool fused_wino_applies(int k, int stride, int dil, int groups, int Cin, int pad, long long tiles)
{
    return k == 3 && stride == 1 && dil == 1 && groups == 1 && Cin % 8 == 0 && pad <= 2 && tiles > 0 &&
           tiles < (1ll << 31) - 64;
}

cudaError_t fused_wino_setup(FusedWino* fw, int Cout, int cin_pad, void* U, const char** why)
{
    fw->ready = false;
    fw->Cout = Cout;
    fw->cin_pad = cin_pad;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&fw->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    // U [16][Cout][cin_pad] TF32-rounded fp32, K-major; box = 32 channels x 128 output channels of one position
    if (!encode_operand_map(&fw->map_u, U, 4, cin_pad, Cout, kPositions, (long long)Cout * cin_pad, kCo)) {
        *why = "cuTensorMapEncodeTiled failed or is unavailable";
        return cudaErrorInvalidValue;
    }
    int stages = (kSmemBudget - 1024 - kVBytes - kStagingBytes) / kUStageBytes;
    if (stages > kMaxUStages) stages = kMaxUStages;
    fw->u_stages = stages;
    fw->smem_bytes = 1024 + kVBytes + stages * kUStageBytes + kStagingBytes;
    e = cudaFuncSetAttribute(fused_f2x2_3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, fw->smem_bytes);
    if (e != cudaSuccess) return e;
    fw->ready = true;
    return cudaSuccess;
}

cudaError_t launch_fused_wino(const FusedWino& fw, const float* x, const float* bias, float* y, const WinoGeom& g, int relu,
                              const TransformMatrices& mats, int* status, cudaStream_t stream)
{
    if (!fw.ready || g.m != 2 || g.k != 3 || g.alpha != 4) return cudaErrorInvalidValue;
    if (g.tiles <= 0) return cudaSuccess;
    wino::MatBt2 bt;
    std::memset(&bt, 0, sizeof(bt));
    for (int i = 0; i < 16; ++i) bt.v[i] = make_float2(mats.Bt[i], mats.Bt[i]);
    MatAt4 at;
    for (int i = 0; i < 8; ++i) at.v[i] = mats.At[i];
    FusedParams p;
    p.x = x; p.bias = bias; p.y = y;
    p.images = g.images; p.Cin = g.Cin; p.Cout = g.Cout; p.H = g.H; p.W = g.W; p.OH = g.OH; p.OW = g.OW; p.pad = g.pad;
    p.th = g.th; p.tw = g.tw; p.relu = relu;
    p.tiles = (int)g.tiles;
    p.n_tile_blocks = (int)((g.tiles + kTiles - 1) / kTiles);
    p.n_co_blocks = (g.Cout + kCo - 1) / kCo;
    p.k_blocks = (g.cin_pad + kKBlock - 1) / kKBlock;
    p.u_stages = fw.u_stages;
    const long long items = (long long)p.n_tile_blocks * p.n_co_blocks;
    if (items >= (1ll << 31)) return cudaErrorInvalidValue;
    p.n_items = (int)items;
    p.sym = wino::bt_has_symmetric_structure(mats.Bt, 4) ? 1 : 0;
    p.status = status;
    const int grid = p.n_items < fw.num_sms ? p.n_items : fw.num_sms;
    return launch_overlapped(fused_f2x2_3x3_kernel, dim3((unsigned)grid), dim3(kThreads), (size_t)fw.smem_bytes, stream,
                             fw.map_u, bt, at, p);
}

}  // namespace mnnb
