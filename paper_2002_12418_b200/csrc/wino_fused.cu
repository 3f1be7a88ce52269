// Winograd F(2x2, 3x3) as ONE kernel (Eq. 6): y = A^T [ sum_c (G w G^T) (.) (B^T d B) ] A + bias, ReLU.
//
// The three stages of Eq. 6 run inside one persistent CTA per SM, so that neither the transformed input V
// nor the products M ever reach HBM (Section 3.3.1 (2) notes that memory access dominates the Hadamard form;
// this removes the two largest tensors from memory altogether):
//   - eight producer warps read the 4 x 4 input windows of a block of 32 tiles, compute B^T d B in registers
//     (packed fp32 pairs, two channels per lane) and write the sixteen transform positions, rounded to TF32,
//     straight into shared memory in the 64-byte-swizzled K-major layout the tensor core reads (two buffers
//     of 16 input channels, so that the transform of the next block overlaps the MMAs of this one);
//   - one thread streams the transformed weights, which were stored at preparation time in exactly the byte
//     order of that shared-memory layout, with plain bulk copies (cp.async.bulk, 32 KB = four transform
//     positions x 128 output channels x 16 input channels per copy) through a ring of four slots;
//   - one thread issues tcgen05.mma (kind::tf32, M = 128 output channels, N = 32 tiles, K = 8 per instruction)
//     into SIXTEEN accumulators, one per transform position, which together fill the 512 columns of tensor
//     memory.  Consecutive MMAs into one accumulator wait for each other, so the K steps of a slot are
//     interleaved across its four accumulators, every descriptor a constant offset from a base;
//   - eight epilogue warps read the sixteen accumulators of their output channels with tcgen05.ld, apply
//     A^T . A, bias and ReLU in registers, transpose through a small staging buffer so that consecutive lanes
//     hold consecutive tiles, and store rows of y.
// A work item is (block of 32 consecutive tiles, block of 128 output channels).  Tensor memory holds exactly
// one item, so the epilogue of an item and the MMAs of the next do not overlap; the producers and the weight
// stream run ahead meanwhile.  Every mbarrier wait is bounded and reports through the status word.
#include "wino_fused.h"

#include <cstring>

#include "umma.cuh"
#include "wino_input.cuh"

namespace mnnb {

namespace {

constexpr int kProducerWarps = 8;
constexpr int kEpilogueWarps = 8;
constexpr int kThreads = 32 * (2 + kEpilogueWarps + kProducerWarps);   // warp 0 weight stream, warp 1 MMA, epilogue, producers
constexpr int kTiles = 32;             // tiles per work item (MMA N)
constexpr int kCo = 128;               // output channels per work item (MMA M)
constexpr int kKBlock = 16;            // input channels per pipeline step: one 64-byte row of TF32
constexpr int kRowBytes = kKBlock * 4;
constexpr int kPositions = 16;         // alpha^2
constexpr int kGroup = 4;              // transform positions per weight copy, interleaved by the MMA thread
constexpr int kGroups = kPositions / kGroup;
constexpr int kSlots = 4;              // ring of weight copies
constexpr int kUPosBytes = kCo * kRowBytes;                 // one transform position of U for one K block: 8 KB
constexpr int kUSlotBytes = kGroup * kUPosBytes;            // one copy: 32 KB
constexpr int kUBlockBytes = kPositions * kUPosBytes;       // all positions of one (channel block, K block): 128 KB
constexpr int kVPosBytes = kTiles * kRowBytes;              // one transform position of V: 2 KB
constexpr int kVBufBytes = kPositions * kVPosBytes;         // 32 KB
constexpr int kVBufs = 2;
constexpr int kRoundTiles = 4;                              // tiles per epilogue round
constexpr int kEpiTiles = kTiles / (kEpilogueWarps / 4);    // tiles per epilogue warp
constexpr int kStageRow = kRoundTiles * 4 + 4;              // staging: 4 outputs per tile and channel, + 4 words of padding
constexpr int kStagingBytes = kEpilogueWarps * 32 * kStageRow * 4;
constexpr int kSmemBytes = 1024 + kVBufs * kVBufBytes + kSlots * kUSlotBytes + kStagingBytes;
static_assert(kSmemBytes <= 226 * 1024, "shared memory budget");

constexpr int kErrStreamWait = 21, kErrMmaWaitU = 22, kErrMmaWaitV = 23, kErrMmaWaitAcc = 24, kErrEpilogueWait = 25,
              kErrProducerWait = 26;

struct MatAt4 { float v[2 * 4]; };     // A^T of F(2, 3): [2][4]
struct MatG43 { float v[4 * 3]; };     // G of F(2, 3): [4][3]

struct FusedParams {
    const float* x;
    const uint8_t* U;        // packed transformed weights
    const float* bias;
    float* y;
    int images, Cin, Cout, H, W, OH, OW, pad, th, tw, relu;
    int tiles;               // images * th * tw
    int n_tile_blocks, n_co_blocks, k_blocks;
    int n_items;
    int sym;                 // B^T has the symmetric-point structure
    int* status;
};

// Byte offset of (row, 16-byte piece) inside a matrix of 64-byte rows stored with the 64-byte swizzle: the four
// pieces of a row are permuted by (row / 2) mod 4 (address bits 4-5 xor bits 7-8).
__host__ __device__ __forceinline__ uint32_t swz64(uint32_t row, uint32_t piece)
{
    return row * 64u + ((piece ^ ((row >> 1) & 3u)) << 4);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Contiguous bulk copy global -> shared memory of this CTA; completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&r)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr)
                 : "memory");
}

// tcgen05.mma kind::tf32 with both shared-memory descriptors given as their low words (start address) over a
// common high word (stride between 8-row groups, version, swizzle mode).
__device__ __forceinline__ void mma_tf32_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .b64 da, db;\n\t"
        ".reg .pred p;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %4, p;\n\t"
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// K-major operand of 64-byte rows, 64-byte swizzle: 8-row groups are 512 bytes apart.
constexpr uint32_t kDescHi = (512u >> 4) | (1u << 14) | (4u << 29);   // stride offset, descriptor version, swizzle mode
constexpr uint32_t kDescLo = 1u << 16;                                // leading offset (unused with a swizzle)

__device__ __forceinline__ float2 tf32_pair(float2 v)
{
    return make_float2(wino::round_tf32_v(v.x), wino::round_tf32_v(v.y));
}

// The 4 x 4 window of one tile for a channel pair (zeros outside the image and beyond Cin).
__device__ __forceinline__ void load_window(float2 (&d)[4][4], const float* p0, size_t plane, int W, unsigned mask, bool c0_ok,
                                            bool c1_ok)
{
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            const bool in = (mask >> (r * 4 + cc)) & 1u;
            const ptrdiff_t off = (ptrdiff_t)r * W + cc;
            d[r][cc].x = (in && c0_ok) ? __ldg(p0 + off) : 0.0f;
            d[r][cc].y = (in && c1_ok) ? __ldg(p0 + plane + off) : 0.0f;
        }
}

__global__ void __launch_bounds__(kThreads, 1)
fused_f2x2_3x3_kernel(const __grid_constant__ wino::MatBt2 Bt, MatAt4 At, FusedParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t u_full[kSlots];
    __shared__ __align__(8) uint64_t u_empty[kSlots];
    __shared__ __align__(8) uint64_t v_full[kVBufs];
    __shared__ __align__(8) uint64_t v_empty[kVBufs];
    __shared__ __align__(8) uint64_t acc_full, acc_empty;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    volatile int* abortp = &abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t v_base = smem_base;                                 // V: [buffer][position][tile][16 channels], swizzled
    const uint32_t u_base = smem_base + kVBufs * kVBufBytes;           // U ring: [slot][position in group][128 rows][16 channels]
    uint8_t* const generic_base = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    float* const staging = reinterpret_cast<float*>(generic_base + kVBufs * kVBufBytes + kSlots * kUSlotBytes);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSlots; ++s) {
            ptx::mbar_init(ptx::smem_u32(&u_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&u_empty[s]), 1);
        }
        for (int s = 0; s < kVBufs; ++s) {
            ptx::mbar_init(ptx::smem_u32(&v_full[s]), kProducerWarps);
            ptx::mbar_init(ptx::smem_u32(&v_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&acc_full), 1);
        ptx::mbar_init(ptx::smem_u32(&acc_empty), kEpilogueWarps);
        abort_flag = 0;
        ptx::fence_barrier_init();
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
        // ------------------------------ weight stream (bulk copies) ------------------------------
        if (lane == 0) {
            uint32_t slot = 0, phase = 0;
            bool ok = true;
            for (int item = first; item < p.n_items && ok; item += step) {
                const int cb = item / p.n_tile_blocks;
                const uint8_t* src = p.U + (size_t)cb * p.k_blocks * kUBlockBytes;
                for (int c = 0; c < p.k_blocks * kGroups; ++c) {           // consecutive copies are consecutive in memory
                    if (!ptx::mbar_wait_relaxed(ptx::smem_u32(&u_empty[slot]), phase ^ 1u, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrStreamWait);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&u_full[slot]);
                    ptx::mbar_expect_tx(bar, kUSlotBytes);
                    bulk_load(u_base + slot * kUSlotBytes, src + (size_t)c * kUSlotBytes, kUSlotBytes, bar);
                    if (++slot == kSlots) {
                        slot = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issue ------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::mma_idesc(2, kCo, kTiles);
            uint32_t slot = 0, phase = 0, buf = 0, v_phase = 0, acc_phase = 0;
            bool ok = true;
            const uint32_t a_lo_base = kDescLo + (u_base >> 4), b_lo_base = kDescLo + (v_base >> 4);
            for (int item = first; item < p.n_items && ok; item += step) {
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&acc_empty), acc_phase ^ 1u, abortp)) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitAcc);
                    *abortp = 1;
                    break;
                }
                ptx::tc_fence_after();
                for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&v_full[buf]), v_phase, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitV);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t acc0 = kb != 0 ? 1u : 0u;
#pragma unroll 1
                    for (int grp = 0; grp < kGroups; ++grp) {
                        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&u_full[slot]), phase, abortp)) {
                            if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitU);
                            *abortp = 1;
                            ok = false;
                            break;
                        }
                        ptx::tc_fence_after();
                        const uint32_t a_lo = a_lo_base + slot * (kUSlotBytes >> 4);
                        const uint32_t b_lo = b_lo_base + buf * (kVBufBytes >> 4) + (uint32_t)grp * ((kGroup * kVPosBytes) >> 4);
                        const uint32_t d_t = tmem_base + (uint32_t)grp * (kGroup * kTiles);
#pragma unroll
                        for (int ks = 0; ks < kKBlock / 8; ++ks)
#pragma unroll
                            for (int g = 0; g < kGroup; ++g)
                                mma_tf32_lo(d_t + g * kTiles, a_lo + g * (kUPosBytes >> 4) + ks * 2,
                                            b_lo + g * (kVPosBytes >> 4) + ks * 2, kDescHi, idesc, ks != 0 ? 1u : acc0);
                        ptx::mma_commit(ptx::smem_u32(&u_empty[slot]));
                        if (++slot == kSlots) {
                            slot = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    ptx::mma_commit(ptx::smem_u32(&v_empty[buf]));     // this buffer may be overwritten once these MMAs retire
                    if (++buf == kVBufs) {
                        buf = 0;
                        v_phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::mma_commit(ptx::smem_u32(&acc_full));
                acc_phase ^= 1u;
            }
        }
    } else if (warp < 2 + kEpilogueWarps) {
        // ------------------------------ epilogue: A^T . A, bias, ReLU, store ------------------------------
        const int q = warp & 3;                                      // quarter of the tensor-memory lanes this warp may read
        const int part = (warp - 2) >> 2;                            // which kEpiTiles tiles of the block this warp handles
        float* const stg = staging + (warp - 2) * 32 * kStageRow;
        uint32_t acc_phase = 0;
        const bool y_pairs = (p.OW % 2 == 0) && ((reinterpret_cast<uintptr_t>(p.y) & 7u) == 0);
        const size_t plane = (size_t)p.OH * p.OW;
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
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(part * kEpiTiles);
#pragma unroll 1
            for (int rd = 0; rd < kEpiTiles / kRoundTiles; ++rd) {
                {
                    uint32_t m[kPositions][4];
#pragma unroll
                    for (int xi = 0; xi < kPositions; ++xi) tmem_ld4(taddr + (uint32_t)(xi * kTiles + rd * kRoundTiles), m[xi]);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int t = 0; t < kRoundTiles; ++t) {
                        // rows: s[a][j] = sum_i At[a][i] M[i][j]; then o[a][c] = sum_j s[a][j] At[c][j]
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
                        *reinterpret_cast<float4*>(stg + lane * kStageRow + t * 4) = make_float4(o[0], o[1], o[2], o[3]);
                    }
                }
                __syncwarp();
                // read back with lanes = (tile j, output row r, channel quarter): rows of y
                {
                    const int j = lane & 3, r = (lane >> 2) & 1, cs = lane >> 3;
                    const int tile = tb * kTiles + part * kEpiTiles + rd * kRoundTiles + j;
                    const bool tile_ok = tile < p.tiles;
                    const int tt = tile_ok ? tile : 0;
                    const int tx = tt % p.tw, rest = tt / p.tw;
                    const int ty = rest % p.th, img = rest / p.th;
                    const int oh = ty * 2 + r, ow = tx * 2;
                    const bool row_ok = tile_ok && oh < p.OH;
                    float* const ybase = p.y + (size_t)img * p.Cout * plane + (size_t)oh * p.OW + ow;
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4) {
                        const int cl = c4 * 4 + cs;
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
        // A warp owns 8 consecutive tiles of the block (lane & 7) and 4 channel pairs of each K block (lane >> 3):
        // the 8-byte stores of a half-warp then fall into distinct banks of the swizzled rows.
        const int pw = warp - 2 - kEpilogueWarps;
        const int t8 = lane & 7, cp4 = lane >> 3;
        const int row = (pw & 3) * 8 + t8;                            // the tile's row in every V[xi] matrix
        const int pair = (pw >> 2) * 4 + cp4;                         // channel pair 0..7 of the K block
        const uint32_t in_buf = swz64((uint32_t)row, (uint32_t)(pair >> 1)) + (uint32_t)((pair & 1) << 3);
        uint32_t buf = 0, v_phase = 0;
        bool ok = true;
        const size_t plane = (size_t)p.H * p.W;
        const int n_local = first < p.n_items ? (p.n_items - first + step - 1) / step : 0;
        const long long n_steps = (long long)n_local * p.k_blocks;    // (item, K block) steps of this CTA
        float2 d[4][4];
        // requests the window of this lane's (tile, channel pair) for step s
        auto step_window = [&](long long s, float2 (&dst)[4][4]) {
            const int li = (int)(s / p.k_blocks), kb = (int)(s - (long long)li * p.k_blocks);
            const int item = first + li * step;
            const int cb = item / p.n_tile_blocks, tb = item - cb * p.n_tile_blocks;
            const int tile = tb * kTiles + row;
            const bool tile_ok = tile < p.tiles;
            const int tt = tile_ok ? tile : 0;
            const int tx = tt % p.tw, rest = tt / p.tw;
            const int ty = rest % p.th, img = rest / p.th;
            const int ih0 = ty * 2 - p.pad, iw0 = tx * 2 - p.pad;
            unsigned mask = 0;
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (tile_ok && ih0 + r >= 0 && ih0 + r < p.H && iw0 + c >= 0 && iw0 + c < p.W) mask |= 1u << (r * 4 + c);
            const int c = kb * kKBlock + pair * 2;
            const float* p0 = p.x + ((ptrdiff_t)((size_t)img * p.Cin + c) * (ptrdiff_t)plane + (ptrdiff_t)ih0 * p.W + iw0);
            load_window(dst, p0, plane, p.W, mask, c < p.Cin, c + 1 < p.Cin);
        };
        if (n_steps > 0) step_window(0, d);
        for (long long s = 0; s < n_steps && ok; ++s) {
            // transform the rows of the window requested one step ago ...
            float2 h[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (p.sym) wino::pass_1d<4, true, float2>(d[r], h[r], Bt);
                else wino::pass_1d<4, false, float2>(d[r], h[r], Bt);
            }
            // ... and request the next one, so that its latency is covered by this step's arithmetic and stores
            if (s + 1 < n_steps) step_window(s + 1, d);
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_relaxed(ptx::smem_u32(&v_empty[buf]), v_phase ^ 1u, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrProducerWait);
                    *abortp = 1;
                }
                ok = false;
                break;
            }
            uint8_t* const dst = generic_base + buf * kVBufBytes + in_buf;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float2 col[4], o[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) col[r] = h[r][j];
                if (p.sym) wino::pass_1d<4, true, float2>(col, o, Bt);
                else wino::pass_1d<4, false, float2>(col, o, Bt);
#pragma unroll
                for (int i = 0; i < 4; ++i) *reinterpret_cast<float2*>(dst + (i * 4 + j) * kVPosBytes) = tf32_pair(o[i]);
            }
            fence_proxy_async_smem();                      // the tensor core reads these through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&v_full[buf]));
            if (++buf == kVBufs) {
                buf = 0;
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

// U = G w G^T for every (output channel, input channel) of the padded ranges, written in the packed layout.
__global__ void fused_weight_transform_kernel(const float* __restrict__ w, uint8_t* __restrict__ U, int Cout, int Cin, int k_blocks,
                                              long long total, MatG43 G)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= total) return;
    const int cin_pad = k_blocks * kKBlock;
    const int ci = (int)(gid % cin_pad), co = (int)(gid / cin_pad);
    float g[9];
    const bool real = ci < Cin && co < Cout;
#pragma unroll
    for (int e = 0; e < 9; ++e) g[e] = real ? w[((size_t)co * Cin + ci) * 9 + e] : 0.0f;
    float t[4][3];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int b = 0; b < 3; ++b) {
            float s = 0.0f;
#pragma unroll
            for (int a = 0; a < 3; ++a) s = fmaf(G.v[i * 3 + a], g[a * 3 + b], s);
            t[i][b] = s;
        }
    const int cb = co / kCo, r = co % kCo, kb = ci / kKBlock, c = ci % kKBlock;
    uint8_t* base = U + ((size_t)cb * k_blocks + kb) * kUBlockBytes + swz64((uint32_t)r, (uint32_t)(c >> 2)) + (c & 3) * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float s = 0.0f;
#pragma unroll
            for (int b = 0; b < 3; ++b) s = fmaf(t[i][b], G.v[j * 3 + b], s);
            *reinterpret_cast<float*>(base + (size_t)(i * 4 + j) * kUPosBytes) = wino::round_tf32_v(s);
        }
}

}  // namespace

bool fused_wino_applies(int k, int stride, int dil, int groups, int pad, long long tiles)
{
    return k == 3 && stride == 1 && dil == 1 && groups == 1 && pad <= 2 && tiles > 0 && tiles < (1ll << 31) - 64;
}

long long fused_wino_weight_bytes(int Cout, int Cin)
{
    const long long co_blocks = (Cout + kCo - 1) / kCo, k_blocks = (Cin + kKBlock - 1) / kKBlock;
    return co_blocks * k_blocks * kUBlockBytes;
}

cudaError_t fused_wino_setup(FusedWino* fw, int Cout, int Cin, const void* U_packed, const char** why)
{
    fw->ready = false;
    if ((reinterpret_cast<uintptr_t>(U_packed) & 15u) != 0) {
        *why = "the packed weights must be 16-byte aligned";
        return cudaErrorInvalidValue;
    }
    fw->U = U_packed;
    fw->Cout = Cout;
    fw->Cin = Cin;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&fw->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    fw->smem_bytes = kSmemBytes;
    e = cudaFuncSetAttribute(fused_f2x2_3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    fw->ready = true;
    return cudaSuccess;
}

cudaError_t launch_fused_wino_weights(const float* w, void* U_packed, int Cout, int Cin, const TransformMatrices& mats,
                                      cudaStream_t stream)
{
    MatG43 G;
    for (int i = 0; i < 12; ++i) G.v[i] = mats.G[i];
    const int co_blocks = (Cout + kCo - 1) / kCo, k_blocks = (Cin + kKBlock - 1) / kKBlock;
    const long long total = (long long)co_blocks * kCo * k_blocks * kKBlock;
    const int threads = 128;
    fused_weight_transform_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, stream>>>(
        w, static_cast<uint8_t*>(U_packed), Cout, Cin, k_blocks, total, G);
    return cudaGetLastError();
}

cudaError_t launch_fused_wino(const FusedWino& fw, const float* x, const float* bias, float* y, const WinoGeom& g, int relu,
                              const TransformMatrices& mats, int* status, cudaStream_t stream)
{
    if (!fw.ready || g.m != 2 || g.k != 3 || g.alpha != 4 || g.Cin != fw.Cin || g.Cout != fw.Cout) return cudaErrorInvalidValue;
    if (g.tiles <= 0) return cudaSuccess;
    wino::MatBt2 bt;
    std::memset(&bt, 0, sizeof(bt));
    for (int i = 0; i < 16; ++i) bt.v[i] = make_float2(mats.Bt[i], mats.Bt[i]);
    MatAt4 at;
    for (int i = 0; i < 8; ++i) at.v[i] = mats.At[i];
    FusedParams p;
    p.x = x; p.U = static_cast<const uint8_t*>(fw.U); p.bias = bias; p.y = y;
    p.images = g.images; p.Cin = g.Cin; p.Cout = g.Cout; p.H = g.H; p.W = g.W; p.OH = g.OH; p.OW = g.OW; p.pad = g.pad;
    p.th = g.th; p.tw = g.tw; p.relu = relu;
    p.tiles = (int)g.tiles;
    p.n_tile_blocks = (int)((g.tiles + kTiles - 1) / kTiles);
    p.n_co_blocks = (g.Cout + kCo - 1) / kCo;
    p.k_blocks = (g.Cin + kKBlock - 1) / kKBlock;
    const long long items = (long long)p.n_tile_blocks * p.n_co_blocks;
    if (items >= (1ll << 31)) return cudaErrorInvalidValue;
    p.n_items = (int)items;
    p.sym = wino::bt_has_symmetric_structure(mats.Bt, 4) ? 1 : 0;
    p.status = status;
    const int grid = p.n_items < fw.num_sms ? p.n_items : fw.num_sms;
    return launch_overlapped(fused_f2x2_3x3_kernel, dim3((unsigned)grid), dim3(kThreads), (size_t)fw.smem_bytes, stream, bt, at,
                             p);
}

}  // namespace mnnb
