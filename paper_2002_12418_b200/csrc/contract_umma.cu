// Batched channel contraction on the 5th-generation tensor cores (Section 3.3.1 (2):
// the Hadamard product of Eq. 6 summed over channels, recast as one matrix product
// per transform position xi):
//     out[xi][co][t] = sum_c U[xi][co][c] * V[xi][t][c]
// A persistent, warp-specialised kernel: one thread feeds shared memory with TMA
// (128-byte-swizzled K-major tiles of V and U), one thread issues tcgen05.mma with
// the accumulator in tensor memory (128 tiles x BN output channels, double
// buffered), four warps drain the accumulator with tcgen05.ld and store it (one per
// quarter of the tensor-memory lanes, the load of the next 16 columns in flight while
// the previous 16 are stored; two warps per quarter, each taking half of the columns,
// gain nothing on long K loops, where the stores already run near the HBM write rate,
// and are used where the K loop is at most two blocks long).
// The MMA "M" dimension is the tile index t (operand A = V), "N" the output channel
// (operand B = U), "K" the input channel; TF32 or BF16 operands, fp32 accumulation;
// with passes = 3 the operands come as hi + lo pairs and hi*hi + lo*hi + hi*lo are
// accumulated.  In tensor memory a lane is a tile and a column an output channel, so
// the 32 lanes of an epilogue warp write 128 contiguous bytes of out[xi][co][.] per
// store: one full line per request.  (With channels on the lanes and 128-bit stores
// the instruction count is lower but every store touches 32 rows; measured slower on
// short K loops, where the epilogue decides.)
//
// A 1x1 stride-1 convolution needs no patch matrix: x[n] = [Cin][H*W] already is operand A, stored with the
// M index (the pixel) contiguous.  In that mode (a_mn) the MMA reads A as an MN-major operand made of
// "atoms" of 32 pixels x 32 channels, and a work item covers up to four consecutive atoms of ONE image, one
// per epilogue warp.  The producer fetches the item's full atoms with a single 4-D box {32 pixels, 32
// channels, n atoms} (x viewed as [image][atom][channel][32 pixels]; one box of 16 KB moves several times
// faster than four boxes of 4 KB) and a ragged last atom of the image with a 3-D box over [image][channel]
// [pixel], whose pixels past H*W read as zeros, so no read leaves x.  Atom slots of the last item of an
// image that hold no atom are not loaded; their accumulator rows are not stored.  The tensor core drops the
// low 13 mantissa bits of the fp32 values it is given (truncation, where the stored operands are rounded
// to nearest).
#include <cuda_bf16.h>

#include "contract_umma.h"
#include "kernels.h"
#include "planner.h"
#include "umma.cuh"

namespace mnnb {

namespace {

// warp 0: TMA, warp 1: MMA + TMEM owner, then 4 or 8 epilogue warps (KernelParams::epi_warps; the warps of a
// lane quarter split the columns).  Eight pay where the K loop is one or two blocks long and the epilogue
// decides (a 32 -> 64 pointwise layer at 112 x 112: 78 -> 68 us); on long K loops they cost 0.3-0.6 %.
constexpr int kMaxEpilogueWarps = 8;
constexpr int kMaxThreads = 64 + 32 * kMaxEpilogueWarps;
constexpr int kTileM = 128;            // tiles (rows of V) per work item
constexpr int kMaxStages = 8;
constexpr int kMaxSharedBias = 2048;    // output channels whose bias is staged in shared memory (+ 16 of slack)
constexpr int kSwizzleBytes = 128;     // bytes of K per shared-memory row
constexpr int kSmemBudget = 200 * 1024;

struct KernelParams {
    int alpha2, n_tile_blocks, n_co_blocks, bn, k_blocks, passes, stages, tmem_cols;   // bn = output channels per work item
    int Cout;
    long long tiles;
    long long n_items;
    ContractEpilogue epi;
    int* status;
    // a_mn mode: operand A comes from x [images][Cin][hw]; atoms of 32 pixels: full_atoms = hw / 32 whole ones
    // and a ragged one when hw % 32 != 0; tiles_per_image work items of up to four atoms cover an image
    int a_mn, hw, full_atoms, atoms_per_image, tiles_per_image;
    // 1: hi and lo operand tiles arrive with one copy each for V and U (maps with a hi / lo dimension, see
    // encode_operand_pair_map); halves the copies the producer issues per stage
    int merged;
    int epi_warps;     // 4 or 8 (the block has 64 + 32 * epi_warps threads)
};

// status codes written on a bounded wait that ran out
constexpr int kErrProducerWait = 1, kErrMmaWaitFull = 2, kErrMmaWaitTmem = 3, kErrEpilogueWait = 4;

// Shared-memory descriptor of a K-major operand tile whose rows are SW bytes long and SW-byte swizzled.
template <int SW>
__device__ __forceinline__ uint64_t desc_k(uint32_t smem_addr)
{
    if (SW == 128) return ptx::smem_desc_k128(smem_addr);
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(512 >> 4) << 32;                         // 8-row groups of 64-byte rows
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)4 << 61;                                  // 64-byte swizzle
    return d;
}

// SW = bytes of K per shared-memory row of an operand tile (the swizzle span): 128, or 64 where 128-byte rows
// would leave room for two pipeline stages only (hi + lo operands with wide channel blocks): the same bytes
// in flight in twice as many stages keep the tensor core fed across the TMA latency.
template <int KIND, int SW>
__global__ void __launch_bounds__(kMaxThreads, 1)
contract_umma_kernel(const __grid_constant__ CUtensorMap map_v_hi, const __grid_constant__ CUtensorMap map_v_lo,
                     const __grid_constant__ CUtensorMap map_u_hi, const __grid_constant__ CUtensorMap map_u_lo,
                     const __grid_constant__ CUtensorMap map_x_ragged, KernelParams p)
// a_mn mode: map_v_hi = 4-D map over x with the box height of an image's leading items, map_v_lo = the same with
// the box height of its last item, map_x_ragged = 3-D map for the ragged atom.
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[kMaxSharedBias + 16];   // GEMM scheme: bias (zeros if none) for the epilogue

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_bytes = kTileM * SW;                            // one V tile (128 tiles)
    const uint32_t b_bytes = (uint32_t)p.bn * SW;                    // one U tile (bn output channels)
    const uint32_t split = p.passes == 3 ? 2u : 1u;
    const uint32_t stage_bytes = (a_bytes + b_bytes) * split;
    // stage layout: [A_hi][A_lo?][B_hi][B_lo?]
    const uint32_t off_a_lo = a_bytes, off_b_hi = a_bytes * split, off_b_lo = a_bytes * split + b_bytes;
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_u32(&tfull_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&tempty_bar[s]), (uint32_t)p.epi_warps);
        }
        abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_v_hi);
        ptx::prefetch_tensormap(&map_u_hi);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), (uint32_t)p.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const bool bias_in_smem = p.epi.mode == 1 && p.Cout <= kMaxSharedBias;
    if (bias_in_smem && warp >= 2) {
        for (int i = threadIdx.x - 64; i < p.Cout; i += 32 * p.epi_warps) s_bias[i] = p.epi.bias ? __ldg(p.epi.bias + i) : 0.0f;
        asm volatile("bar.sync 1, %0;" ::"r"(32 * p.epi_warps) : "memory");             // the epilogue warps only
    }

    const int k_elems = (KIND == 0 ? 32 : 64) * SW / 128;   // elements of K per shared-memory row

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const int tb = (int)(item % p.n_tile_blocks);
                const long long r = item / p.n_tile_blocks;
                const int nb = (int)(r % p.n_co_blocks);
                const int xi = (int)(r / p.n_co_blocks);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&empty_bar[stage]), phase ^ 1u, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrProducerWait);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&full_bar[stage]);
                    const uint32_t sbase = smem_base + stage * stage_bytes;
                    if (p.a_mn) {
                        const int img = tb / p.tiles_per_image;
                        const int a0 = (tb - img * p.tiles_per_image) * (kTileM / 32);       // first atom of the item
                        const int n_full = min(kTileM / 32, max(0, p.full_atoms - a0));
                        const bool ragged = p.full_atoms < p.atoms_per_image && a0 + kTileM / 32 >= p.atoms_per_image;
                        ptx::mbar_expect_tx(bar, (uint32_t)(n_full + (ragged ? 1 : 0)) * 4096u + b_bytes);
                        if (n_full > 0)
                            ptx::tma_load_4d(sbase, a0 + kTileM / 32 <= p.full_atoms ? &map_v_hi : &map_v_lo, bar, 0,
                                             kb * k_elems, a0, img);
                        if (ragged)
                            ptx::tma_load_3d(sbase + (uint32_t)n_full * 4096u, &map_x_ragged, bar, p.full_atoms * 32,
                                             kb * k_elems, img);
                    } else {
                        ptx::mbar_expect_tx(bar, stage_bytes);
                        if (p.merged) ptx::tma_load_4d(sbase, &map_v_hi, bar, kb * k_elems, tb * kTileM, 0, xi);
                        else ptx::tma_load_3d(sbase, &map_v_hi, bar, kb * k_elems, tb * kTileM, xi);
                    }
                    if (p.merged) {
                        ptx::tma_load_4d(sbase + off_b_hi, &map_u_hi, bar, kb * k_elems, nb * p.bn, 0, xi);
                    } else {
                        ptx::tma_load_3d(sbase + off_b_hi, &map_u_hi, bar, kb * k_elems, nb * p.bn, xi);
                        if (split == 2) {
                            ptx::tma_load_3d(sbase + off_a_lo, &map_v_lo, bar, kb * k_elems, tb * kTileM, xi);
                            ptx::tma_load_3d(sbase + off_b_lo, &map_u_lo, bar, kb * k_elems, nb * p.bn, xi);
                        }
                    }
                    if (++stage == (uint32_t)p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = ptx::mma_idesc(KIND == 0 ? 2 : 1, kTileM, p.bn, p.a_mn != 0);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, abortp)) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitTmem);
                    *abortp = 1;
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.bn;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&full_bar[stage]), phase, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitFull);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t sbase = smem_base + stage * stage_bytes;
#pragma unroll
                    for (int ks = 0; ks < SW / 32; ++ks) {
                        // K-major: 8 K elements are 32 bytes along the row; MN-major: 8 rows of 128 bytes
                        const uint64_t a_hi = (SW == 128 && p.a_mn) ? ptx::smem_desc_mn128_b32(sbase + ks * 1024, 4096)
                                                                    : desc_k<SW>(sbase + ks * 32);
                        const uint64_t b_hi = desc_k<SW>(sbase + off_b_hi + ks * 32);
                        ptx::mma_ss<KIND>(d_tmem, a_hi, b_hi, idesc, (kb | ks) != 0 ? 1u : 0u);
                        if (split == 2) {
                            const uint64_t a_lo = desc_k<SW>(sbase + off_a_lo + ks * 32);
                            const uint64_t b_lo = desc_k<SW>(sbase + off_b_lo + ks * 32);
                            ptx::mma_ss<KIND>(d_tmem, a_lo, b_hi, idesc, 1u);
                            ptx::mma_ss<KIND>(d_tmem, a_hi, b_lo, idesc, 1u);
                        }
                    }
                    ptx::mma_commit(ptx::smem_u32(&empty_bar[stage]));     // stage reusable once these MMAs retire
                    if (++stage == (uint32_t)p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::mma_commit(ptx::smem_u32(&tfull_bar[acc]));           // accumulator complete
                acc ^= 1u;
                if (acc == 0) acc_phase ^= 1u;
            }
        }
    } else {
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int part = (warp - 2) >> 2;             // which part of the columns this warp drains
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (long long item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            const int tb = (int)(item % p.n_tile_blocks);
            const long long r = item / p.n_tile_blocks;
            const int nb = (int)(r % p.n_co_blocks);
            const int xi = (int)(r / p.n_co_blocks);
            // one lane polls for the warp
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_bounded(ptx::smem_u32(&tfull_bar[acc]), acc_phase, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrEpilogueWait);
                    *abortp = 1;
                }
                ok = false;
                break;
            }
            ptx::tc_fence_after();
            const long long t = (long long)tb * kTileM + q * 32 + lane;      // this thread's tile (or GEMM column)
            bool t_ok = t < p.tiles;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * (uint32_t)p.bn;
            const int co0 = nb * p.bn;
            const int n_co = min(p.bn, p.Cout - co0);                        // valid output channels of this item
            // destination of channel co0 for this thread, and the distance to the next channel
            float* dst;
            long long step;
            if (p.epi.mode == 0) {
                step = p.epi.m_row_stride;
                dst = p.epi.M + ((size_t)xi * p.Cout + co0) * p.epi.m_row_stride + t;
            } else if (p.a_mn) {
                const int img = tb / p.tiles_per_image;
                const int pix = ((tb - img * p.tiles_per_image) * (kTileM / 32) + q) * 32 + lane;   // this warp's atom
                t_ok = pix < p.hw;
                step = p.hw;
                dst = p.epi.y + ((size_t)(t_ok ? img : 0) * p.Cout + co0) * p.hw + (t_ok ? pix : 0);
            } else {
                const long long img = t_ok ? t / p.epi.ohw : 0;
                step = p.epi.ohw;
                dst = p.epi.y + ((size_t)img * p.Cout + co0) * p.epi.ohw + (t_ok ? t - img * p.epi.ohw : 0);
            }
            // this warp's chunks of 16 columns
            const int kParts = p.epi_warps >> 2;
            const int n_chunks = (n_co + 15) >> 4;
            const int per_part = (n_chunks + kParts - 1) / kParts;
            const int ch_begin = min(part * per_part, n_chunks), ch_end = min(ch_begin + per_part, n_chunks);
            dst += (long long)ch_begin * 16 * step;
            const bool relu = p.epi.relu != 0;
            auto store_chunk = [&](const uint32_t (&v)[16], int ch) {
                if (!t_ok) return;
                const int c0 = ch * 16;
                const int n = min(16, n_co - c0);
                float* pj = dst;                                   // walks the 16 channels of this chunk
                if (p.epi.mode == 0) {
                    if (n == 16) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            *pj = __uint_as_float(v[j]);
                            pj += step;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (j < n) *pj = __uint_as_float(v[j]);
                            pj += step;
                        }
                    }
                } else {
                    float bz[16];
                    if (bias_in_smem) {
                        // (reads past Cout stay inside the array and are not used)
                        const float4* bp = reinterpret_cast<const float4*>(s_bias + co0 + c0);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float4 q4 = bp[j];
                            bz[4 * j] = q4.x; bz[4 * j + 1] = q4.y; bz[4 * j + 2] = q4.z; bz[4 * j + 3] = q4.w;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) bz[j] = (p.epi.bias && j < n) ? __ldg(p.epi.bias + co0 + c0 + j) : 0.0f;
                    }
                    if (n == 16) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float o = __uint_as_float(v[j]) + bz[j];
                            *pj = relu ? fmaxf(o, 0.0f) : o;
                            pj += step;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float o = __uint_as_float(v[j]) + bz[j];
                            if (j < n) *pj = relu ? fmaxf(o, 0.0f) : o;
                            pj += step;
                        }
                    }
                }
            };
            uint32_t va[16], vb[16];
            if (ch_begin < ch_end) ptx::tmem_ld16(taddr + (uint32_t)(ch_begin * 16), va);
            for (int ch = ch_begin; ch < ch_end; ch += 2) {
                ptx::tmem_ld_wait();
                if (ch + 1 < ch_end) ptx::tmem_ld16(taddr + (uint32_t)((ch + 1) * 16), vb);
                store_chunk(va, ch);
                dst += 16 * step;
                if (ch + 1 < ch_end) {
                    ptx::tmem_ld_wait();
                    if (ch + 2 < ch_end) ptx::tmem_ld16(taddr + (uint32_t)((ch + 2) * 16), va);
                    store_chunk(vb, ch + 1);
                    dst += 16 * step;
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&tempty_bar[acc]));
            acc ^= 1u;
            if (acc == 0) acc_phase ^= 1u;
        }
    }

    // Teardown.  After an aborted run give copies still in flight time to land before the CTA's
    // shared memory is released.
    if (*abortp) __nanosleep(200000);
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// A barrier nobody arrives on: the bounded wait must give up and let the kernel return.
__global__ void wait_probe_kernel(int* word)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int never_set;
    if (threadIdx.x == 0) {
        never_set = 0;
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        ptx::fence_barrier_init();
        *word = 1;
        __threadfence();
        const bool done = ptx::mbar_wait_bounded(ptx::smem_u32(&bar), 0u, &never_set);
        *word = done ? 3 : 2;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    // looked up once; the initialisation of a function-local static is thread-safe
    static const EncodeTiledFn fn = [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(sym);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

}  // namespace

// 3-D map over [planes][rows][k] (k contiguous), box = [1][box_rows][128 bytes of k], 128-byte swizzle.
bool encode_operand_map_sw(CUtensorMap* map, void* base, int elem_bytes, long long k_len, long long rows, long long planes,
                           long long plane_stride_elems, int box_rows, int sw);

bool encode_operand_map(CUtensorMap* map, void* base, int elem_bytes, long long k_len, long long rows, long long planes,
                        long long plane_stride_elems, int box_rows)
{
    return encode_operand_map_sw(map, base, elem_bytes, k_len, rows, planes, plane_stride_elems, box_rows, kSwizzleBytes);
}

// The same with rows of `sw` bytes (128 or 64) and the matching swizzle.
bool encode_operand_map_sw(CUtensorMap* map, void* base, int elem_bytes, long long k_len, long long rows, long long planes,
                           long long plane_stride_elems, int box_rows, int sw)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)k_len, (cuuint64_t)rows, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {(cuuint64_t)k_len * elem_bytes, (cuuint64_t)plane_stride_elems * elem_bytes};
    const cuuint32_t box[3] = {(cuuint32_t)(sw / elem_bytes), (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    CUresult r = fn(map, dt, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    sw == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 4-D map over a hi / lo operand pair: [planes][hi, lo][rows][k], the lo array `lo_offset_bytes` behind the hi
// array; box = [1][2][box_rows][sw bytes of k].  One copy lands the hi tile and, right behind it, the lo tile.
bool encode_operand_pair_map(CUtensorMap* map, void* base_hi, long long lo_offset_bytes, int elem_bytes, long long k_len,
                             long long rows, long long planes, long long plane_stride_elems, int box_rows, int sw)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || lo_offset_bytes <= 0 || lo_offset_bytes % 16 != 0 || lo_offset_bytes >= (1ll << 40)) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)k_len, (cuuint64_t)rows, 2, (cuuint64_t)planes};
    const cuuint64_t strides[3] = {(cuuint64_t)k_len * elem_bytes, (cuuint64_t)lo_offset_bytes,
                                   (cuuint64_t)plane_stride_elems * elem_bytes};
    const cuuint32_t box[4] = {(cuuint32_t)(sw / elem_bytes), (cuuint32_t)box_rows, 2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return fn(map, dt, 4, base_hi, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              sw == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace wino {
// Tensor map over x [images][C][H][W] (fp32) for the input transform's row copies, no swizzle; elements
// outside the tensor read as zero.  Needs W * 4 to be a multiple of 16 bytes and a 16-byte aligned base.
//   split_parity = false: 4-D {W, H, C, images}, box {box_w, 1, 64, 1}: 64 consecutive channels of one row.
//   split_parity = true (C even): 5-D {W, H, 2, C/2, images}, box {box_w, 1, 1, 32, 1}: 32 channels of one
//   parity (c = 2 * pair + parity) of one row.
bool encode_input_map(CUtensorMap* map, const float* x, int images, int C, int H, int W, int box_w, bool split_parity)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || box_w > 256 || (W % 4) != 0 || (box_w % 4) != 0) return false;
    const cuuint64_t plane = (cuuint64_t)H * W * 4;
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r;
    if (split_parity) {
        if (C % 2) return false;
        const cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, 2, (cuuint64_t)(C / 2), (cuuint64_t)images};
        const cuuint64_t strides[4] = {(cuuint64_t)W * 4, plane, 2 * plane, (cuuint64_t)C * plane};
        const cuuint32_t box[5] = {(cuuint32_t)box_w, 1, 1, 32, 1};
        r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)images};
        const cuuint64_t strides[3] = {(cuuint64_t)W * 4, plane, (cuuint64_t)C * plane};
        const cuuint32_t box[4] = {(cuuint32_t)box_w, 1, 64, 1};
        r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    return r == CUDA_SUCCESS;
}
}  // namespace wino

cudaError_t launch_wait_probe(int* device_word, cudaStream_t stream)
{
    wait_probe_kernel<<<1, 32, 0, stream>>>(device_word);
    return cudaGetLastError();
}

cudaError_t umma_contract_setup(UmmaContract* uc, int mode, int alpha2, int Cout, int cin_pad, long long tiles_capacity,
                                void* U_hi, void* U_lo, void* V_hi, void* V_lo, const char** why)
{
    uc->ready = false;
    uc->a_mn = V_hi == nullptr;        // operand A is read from x at launch time (umma_contract_setup_x)
    if (uc->a_mn && (mode != STORE_TF32 || alpha2 != 1)) {
        *why = "reading x as operand A needs single-pass TF32 and one transform position";
        return cudaErrorInvalidValue;
    }
    if (mode == STORE_FP32) {
        *why = "the tensor-core contraction needs TF32 or BF16 operands";
        return cudaErrorInvalidValue;
    }
    const int eb = store_elem_bytes(mode);
    uc->kind = eb == 2 ? 1 : 0;
    uc->passes = store_is_split(mode) ? 3 : 1;
    uc->alpha2 = alpha2;
    uc->Cout = Cout;
    uc->cin_pad = cin_pad;
    uc->tiles_capacity = tiles_capacity;
    if (((long long)cin_pad * eb) % 16 != 0) {
        *why = "operand rows must be a multiple of 16 bytes";
        return cudaErrorInvalidValue;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&uc->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    // output channels per work item (MMA N) and the channel blocks
    contract_tiling((tiles_capacity + kTileM - 1) / kTileM, alpha2, Cout, uc->num_sms, &uc->bn, &uc->n_co_blocks);
    const int split = uc->passes == 3 ? 2 : 1;
    // rows of 128 bytes unless that leaves fewer than three stages and the K loop is long (at least four
    // 128-byte blocks; measured: 512 channels BF16 hi + lo 0.604 -> 0.576 ms, shorter loops lose)
    int sw = kSwizzleBytes;
    if (!uc->a_mn && (kSmemBudget - 1024) / ((kTileM + uc->bn) * sw * split) < 3 && cin_pad * eb >= 4 * sw) sw = 64;
    uc->stages_sw = sw;
    const int k_elems = sw / eb;
    uc->k_blocks = (cin_pad + k_elems - 1) / k_elems;
    const int stage_bytes = (kTileM * sw + uc->bn * sw) * split;
    int stages = (kSmemBudget - 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) {
        *why = "shared memory cannot hold two pipeline stages";
        return cudaErrorInvalidValue;
    }
    uc->stages = stages;
    // Always ask for the full budget so that at most one CTA is resident per SM: a second CTA could
    // otherwise block inside the tensor-memory allocation.
    uc->smem_bytes = kSmemBudget;
    int cols = 32;
    while (cols < 2 * uc->bn) cols *= 2;
    uc->tmem_cols = cols;

    const long long u_plane = (long long)Cout * cin_pad, v_plane = tiles_capacity * cin_pad;
    bool ok = (uc->a_mn || encode_operand_map_sw(&uc->map_v_hi, V_hi, eb, cin_pad, tiles_capacity, alpha2, v_plane, kTileM, sw)) &&
              encode_operand_map_sw(&uc->map_u_hi, U_hi, eb, cin_pad, Cout, alpha2, u_plane, uc->bn, sw);
    if (ok && split == 2)
        ok = encode_operand_map_sw(&uc->map_v_lo, V_lo, eb, cin_pad, tiles_capacity, alpha2, v_plane, kTileM, sw) &&
             encode_operand_map_sw(&uc->map_u_lo, U_lo, eb, cin_pad, Cout, alpha2, u_plane, uc->bn, sw);
    if (!ok) {
        *why = "cuTensorMapEncodeTiled failed or is unavailable";
        return cudaErrorInvalidValue;
    }
    // hi + lo operands that lie in one allocation each (lo behind hi): one copy per operand and stage
    uc->merged = 0;
    if (split == 2 && !uc->a_mn) {
        const long long dv = static_cast<char*>(V_lo) - static_cast<char*>(V_hi), du = static_cast<char*>(U_lo) - static_cast<char*>(U_hi);
        CUtensorMap mv, mu;
        if (encode_operand_pair_map(&mv, V_hi, dv, eb, cin_pad, tiles_capacity, alpha2, v_plane, kTileM, sw) &&
            encode_operand_pair_map(&mu, U_hi, du, eb, cin_pad, Cout, alpha2, u_plane, uc->bn, sw)) {
            uc->map_v_hi = mv;
            uc->map_u_hi = mu;
            uc->merged = 1;
        }
    }
    if (uc->a_mn) uc->map_v_hi = uc->map_u_hi;      // replaced by the map over x at every launch
    if (split == 1) {
        uc->map_v_lo = uc->map_v_hi;
        uc->map_u_lo = uc->map_u_hi;
    }
    for (auto kern : {contract_umma_kernel<0, 128>, contract_umma_kernel<1, 128>, contract_umma_kernel<0, 64>,
                      contract_umma_kernel<1, 64>}) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
    }
    uc->ready = true;
    return cudaSuccess;
}

cudaError_t umma_contract_setup_x(UmmaContract* uc, int Cout, int Cin, int cin_pad, int images, int hw, void* U,
                                  const char** why)
{
    if (hw < 32 || hw % 4 != 0) {
        *why = "reading x as operand A needs H*W >= 32 and a multiple of 4";
        return cudaErrorInvalidValue;
    }
    const int atoms = (hw + 31) / 32, tiles_per_image = (atoms + kTileM / 32 - 1) / (kTileM / 32);
    cudaError_t e = umma_contract_setup(uc, STORE_TF32, 1, Cout, cin_pad, (long long)images * tiles_per_image * kTileM, U,
                                        nullptr, nullptr, nullptr, why);
    if (e != cudaSuccess) return e;
    uc->x_images = images;
    uc->x_cin = Cin;
    uc->x_hw = hw;
    uc->k_blocks = (Cin + 31) / 32;
    return cudaSuccess;
}

cudaError_t launch_contract_umma_x(const UmmaContract& uc, const float* x, const ContractEpilogue& epi, int* status,
                                   cudaStream_t stream)
{
    if (!uc.ready || !uc.a_mn) return cudaErrorInvalidValue;
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return cudaErrorInvalidValue;
    KernelParams p;
    p.a_mn = 1;
    p.merged = 0;
    p.hw = uc.x_hw;
    p.full_atoms = uc.x_hw / 32;
    p.atoms_per_image = (uc.x_hw + 31) / 32;
    p.tiles_per_image = (p.atoms_per_image + kTileM / 32 - 1) / (kTileM / 32);
    // Tensor maps over x, 128-byte swizzle with a 32-byte base.  Whole atoms: x as [image][atom][channel][32
    // pixels] (the atom stride, 128 bytes, is smaller than the channel stride), box = 32 pixels x 32 channels x
    // h atoms, h = 4 for the leading items of an image and what is left for its last item.  Ragged atom: x as
    // [image][channel][pixel], box = 32 pixels x 32 channels, pixels past hw read as zeros.
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const cuuint64_t plane = (cuuint64_t)uc.x_hw * 4;
    auto encode_atoms = [&](CUtensorMap* m, int h) {
        const cuuint64_t dims[4] = {32, (cuuint64_t)uc.x_cin, (cuuint64_t)p.full_atoms, (cuuint64_t)uc.x_images};
        const cuuint64_t strides[3] = {plane, 128, (cuuint64_t)uc.x_cin * plane};
        const cuuint32_t box[4] = {32, 32, (cuuint32_t)h, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(x), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    CUtensorMap map_lead, map_last, map_ragged;
    const int h_lead = p.full_atoms < kTileM / 32 ? p.full_atoms : kTileM / 32;
    int h_last = p.full_atoms - (p.tiles_per_image - 1) * (kTileM / 32);       // whole atoms of an image's last item
    if (h_last < 1 || h_last > kTileM / 32) h_last = h_lead;                   // (none: the map is not used)
    if (!encode_atoms(&map_lead, h_lead) || !encode_atoms(&map_last, h_last)) return cudaErrorInvalidValue;
    {
        const cuuint64_t dims[3] = {(cuuint64_t)uc.x_hw, (cuuint64_t)uc.x_cin, (cuuint64_t)uc.x_images};
        const cuuint64_t strides[2] = {plane, (cuuint64_t)uc.x_cin * plane};
        const cuuint32_t box[3] = {32, 32, 1};
        if (fn(&map_ragged, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    if ((long long)uc.x_images * p.tiles_per_image > 2147483647ll) return cudaErrorInvalidValue;
    p.alpha2 = 1;
    p.n_tile_blocks = uc.x_images * p.tiles_per_image;
    p.n_co_blocks = uc.n_co_blocks;
    p.bn = uc.bn;
    p.k_blocks = uc.k_blocks;
    p.passes = 1;
    p.stages = uc.stages;
    p.tmem_cols = uc.tmem_cols;
    p.Cout = uc.Cout;
    p.tiles = (long long)p.n_tile_blocks * kTileM;
    p.n_items = (long long)p.n_tile_blocks * p.n_co_blocks;
    p.epi = epi;
    p.status = status;
    const long long grid = p.n_items < uc.num_sms ? p.n_items : uc.num_sms;
    p.epi_warps = uc.k_blocks <= 2 ? 8 : 4;
    return launch_overlapped(contract_umma_kernel<0, 128>, dim3((unsigned)grid), dim3(64 + 32 * p.epi_warps), (size_t)uc.smem_bytes, stream,
                             map_lead, map_last, uc.map_u_hi, uc.map_u_lo, map_ragged, p);
}

cudaError_t launch_contract_umma(const UmmaContract& uc, long long tiles, const ContractEpilogue& epi, int* status,
                                 cudaStream_t stream)
{
    if (!uc.ready || uc.a_mn) return cudaErrorInvalidValue;
    if (tiles <= 0) return cudaSuccess;
    if (tiles > uc.tiles_capacity) return cudaErrorInvalidValue;
    KernelParams p;
    p.a_mn = 0;
    p.merged = uc.merged;
    p.hw = 0;
    p.full_atoms = 0;
    p.atoms_per_image = 1;
    p.tiles_per_image = 1;
    p.alpha2 = uc.alpha2;
    p.n_tile_blocks = (int)((tiles + kTileM - 1) / kTileM);
    p.n_co_blocks = uc.n_co_blocks;
    p.bn = uc.bn;
    p.k_blocks = uc.k_blocks;
    p.passes = uc.passes;
    p.stages = uc.stages;
    p.tmem_cols = uc.tmem_cols;
    p.Cout = uc.Cout;
    p.tiles = tiles;
    p.n_items = (long long)p.n_tile_blocks * p.n_co_blocks * uc.alpha2;
    p.epi = epi;
    p.status = status;
    long long grid = p.n_items < uc.num_sms ? p.n_items : uc.num_sms;
    auto kern = uc.kind == 0 ? (uc.stages_sw == 64 ? contract_umma_kernel<0, 64> : contract_umma_kernel<0, 128>)
                             : (uc.stages_sw == 64 ? contract_umma_kernel<1, 64> : contract_umma_kernel<1, 128>);
    p.epi_warps = (uc.alpha2 == 1 && uc.k_blocks <= 2) ? 8 : 4;
    return launch_overlapped(kern, dim3((unsigned)grid), dim3(64 + 32 * p.epi_warps), (size_t)uc.smem_bytes, stream, uc.map_v_hi,
                             uc.map_v_lo, uc.map_u_hi, uc.map_u_lo, uc.map_u_hi, p);
}

}  // namespace mnnb
