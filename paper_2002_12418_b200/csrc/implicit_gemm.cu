// Implicit GEMM: the GEMM scheme for k > 1 strided / dilated / padded layers without a patch matrix.
//
// The product is  y[t][co] = sum_kk patch(t)[kk] U[co][kk]  with t the flat output position (n, oh, ow) and
// kk = (ci * k + a) * k + b.  A persistent CTA per SM:
//   - eight producer warps build the left operand tile (128 output positions x 32 patch elements, TF32) of every
//     pipeline stage themselves: a lane owns one output position for the whole work item and gathers four runs
//     of four consecutive patch elements per stage with plain loads (coalesced across the lanes: neighbouring
//     lanes are neighbouring output positions), rounds them to TF32 and writes them as 16-byte pieces into the
//     128-byte-swizzled K-major layout the tensor core reads.  The loads of the next stage are issued two stages
//     ahead;
//   - one thread fetches the weight tile (bn output channels x 32 patch elements) of every stage with TMA;
//   - one thread issues tcgen05.mma (kind::tf32, M = 128 positions, N = bn channels), accumulators double
//     buffered in tensor memory;
//   - four epilogue warps drain an accumulator, add the bias, apply ReLU and store y (a tensor-memory lane is an
//     output position, so a warp store writes 128 contiguous bytes of one channel plane).
// A tiled TMA copy cannot gather the patches: it would have to start at x offsets (- pad + b * dilation) that are
// not multiples of 16 bytes.  Every mbarrier wait is bounded and reports through the status word.
#include "implicit_gemm.h"

#include "contract_umma.h"
#include "planner.h"
#include "umma.cuh"

namespace mnnb {

namespace {

constexpr int kProducerWarps = 8;
constexpr int kEpilogueWarps = 4;
constexpr int kThreads = 32 * (2 + kEpilogueWarps + kProducerWarps);
constexpr int kTileM = 128;            // output positions per work item
constexpr int kKBlock = 32;            // patch elements per stage: one 128-byte row of TF32
constexpr int kABytes = kTileM * 128;
constexpr int kMaxStages = 6;
constexpr int kSmemBudget = 200 * 1024;
constexpr int kMaxSharedBias = 2048;

constexpr int kErrTmaWait = 31, kErrMmaWaitFull = 32, kErrMmaWaitTmem = 33, kErrEpilogueWait = 34, kErrProducerWait = 35;

struct IgParams {
    const float* x;
    const float* bias;
    float* y;
    int N, Cin, H, W, OH, OW, k, stride, pad, dil, Cout;
    int Kd;                  // Cin * k * k
    long long T;             // N * OH * OW
    int n_tile_blocks, n_co_blocks, bn, k_blocks, stages, tmem_cols;
    long long n_items;
    int relu;
    int tap_major;           // patch elements ordered (a, b, ci) instead of (ci, a, b): a stage is 32 channels of one tap
    int* status;
};

__device__ __forceinline__ float round_tf32(float v)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
implicit_gemm_kernel(const __grid_constant__ CUtensorMap map_u, IgParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[kMaxSharedBias + 16];
    volatile int* abortp = &abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const generic_base = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t b_bytes = (uint32_t)p.bn * 128u;
    const uint32_t stage_bytes = kABytes + b_bytes;                   // [A: 128 x 128 B][B: bn x 128 B]

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1 + kProducerWarps);      // the TMA's expect_tx arrival + the producers
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_u32(&tfull_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&tempty_bar[s]), kEpilogueWarps);
        }
        abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_u);
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
    const bool bias_in_smem = p.Cout <= kMaxSharedBias;
    if (bias_in_smem && warp >= 2 && warp < 2 + kEpilogueWarps) {
        for (int i = threadIdx.x - 64; i < p.Cout; i += 32 * kEpilogueWarps) s_bias[i] = p.bias ? __ldg(p.bias + i) : 0.0f;
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpilogueWarps) : "memory");          // the epilogue warps only
    }

    if (warp == 0) {
        // ------------------------------ weight tiles (TMA) ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const int nb = (int)(item / p.n_tile_blocks);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!ptx::mbar_wait_relaxed(ptx::smem_u32(&empty_bar[stage]), phase ^ 1u, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrTmaWait);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t bar = ptx::smem_u32(&full_bar[stage]);
                    ptx::mbar_expect_tx(bar, b_bytes);
                    ptx::tma_load_3d(smem_base + stage * stage_bytes + kABytes, &map_u, bar, kb * kKBlock, nb * p.bn, 0);
                    if (++stage == (uint32_t)p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issue ------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::mma_idesc(2, kTileM, p.bn);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, abortp)) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrMmaWaitTmem);
                    *abortp = 1;
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
                    for (int ks = 0; ks < 4; ++ks)
                        ptx::mma_ss<0>(d_tmem, ptx::smem_desc_k128(sbase + ks * 32), ptx::smem_desc_k128(sbase + kABytes + ks * 32),
                                       idesc, (kb | ks) != 0 ? 1u : 0u);
                    ptx::mma_commit(ptx::smem_u32(&empty_bar[stage]));
                    if (++stage == (uint32_t)p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::mma_commit(ptx::smem_u32(&tfull_bar[acc]));
                acc ^= 1u;
                if (acc == 0) acc_phase ^= 1u;
            }
        }
    } else if (warp < 2 + kEpilogueWarps) {
        // ------------------------------ epilogue: bias, ReLU, store y ------------------------------
        const int q = warp & 3;                       // quarter of the tensor-memory lanes this warp may read
        const long long ohw = (long long)p.OH * p.OW;
        uint32_t acc = 0, acc_phase = 0;
        const bool relu = p.relu != 0;
        for (long long item = blockIdx.x; item < p.n_items; item += gridDim.x) {
            const int tb = (int)(item % p.n_tile_blocks);
            const int nb = (int)(item / p.n_tile_blocks);
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_relaxed(ptx::smem_u32(&tfull_bar[acc]), acc_phase, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrEpilogueWait);
                    *abortp = 1;
                }
                break;
            }
            ptx::tc_fence_after();
            const long long t = (long long)tb * kTileM + q * 32 + lane;      // this lane's output position
            const bool t_ok = t < p.T;
            const long long img = t_ok ? t / ohw : 0;
            const int co0 = nb * p.bn;
            const int n_co = min(p.bn, p.Cout - co0);
            float* dst = p.y + ((size_t)img * p.Cout + co0) * ohw + (t_ok ? t - img * ohw : 0);
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * (uint32_t)p.bn;
            const int n_chunks = (n_co + 15) >> 4;
            auto store_chunk = [&](const uint32_t (&v)[16], int ch) {
                if (!t_ok) return;
                const int c0 = ch * 16;
                const int n = min(16, n_co - c0);
                float bz[16];
                if (bias_in_smem) {
                    const float4* bp = reinterpret_cast<const float4*>(s_bias + co0 + c0);   // (reads past Cout stay inside the array)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 q4 = bp[j];
                        bz[4 * j] = q4.x; bz[4 * j + 1] = q4.y; bz[4 * j + 2] = q4.z; bz[4 * j + 3] = q4.w;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) bz[j] = (p.bias && j < n) ? __ldg(p.bias + co0 + c0 + j) : 0.0f;
                }
                float* pj = dst + (long long)c0 * ohw;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float o = __uint_as_float(v[j]) + bz[j];
                    if (j < n) *pj = relu ? fmaxf(o, 0.0f) : o;
                    pj += ohw;
                }
            };
            uint32_t va[16], vb[16];
            if (n_chunks > 0) ptx::tmem_ld16(taddr, va);
            for (int ch = 0; ch < n_chunks; ch += 2) {
                ptx::tmem_ld_wait();
                if (ch + 1 < n_chunks) ptx::tmem_ld16(taddr + (uint32_t)((ch + 1) * 16), vb);
                store_chunk(va, ch);
                if (ch + 1 < n_chunks) {
                    ptx::tmem_ld_wait();
                    if (ch + 2 < n_chunks) ptx::tmem_ld16(taddr + (uint32_t)((ch + 2) * 16), va);
                    store_chunk(vb, ch + 1);
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&tempty_bar[acc]));
            acc ^= 1u;
            if (acc == 0) acc_phase ^= 1u;
        }
    } else {
        // ------------------------------ producers: the patch tile of every stage ------------------------------
        // A lane owns one output position (row of the tile) and, per stage, 16 consecutive patch elements
        // (four 16-byte pieces): rows (pw & 3) * 32 + lane, pieces (pw >> 2) * 4 .. + 3.  The eight lanes of a
        // quarter-warp write the same piece index of eight consecutive rows, which the swizzle spreads over
        // all banks.
        const int pw = warp - 2 - kEpilogueWarps;
        const int row = (pw & 3) * 32 + lane;
        const int piece0 = (pw >> 2) * 4;
        const int k2 = p.k * p.k;
        const long long ohw = (long long)p.OH * p.OW;
        const size_t plane = (size_t)p.H * p.W;
        const unsigned first = blockIdx.x;
        const long long n_local = (long long)first < p.n_items ? (p.n_items - first + gridDim.x - 1) / gridDim.x : 0;
        const long long n_steps = n_local * p.k_blocks;
        uint32_t stage = 0, phase = 0;
        float va[16], vb[16];                               // the patch elements of the next two steps, in flight
        // The gather stream: steps are taken in order, so a cursor (work item, K block) advances by one per call and
        // the decode of the lane's output position is redone only when the work item changes.
        long long cur_item = first;
        int cur_kb = 0;
        const float* base = p.x;
        unsigned rows_in = 0, cols_in = 0;
        auto decode_item = [&]() {
            const int tb = (int)(cur_item % p.n_tile_blocks);
            const int t = tb * kTileM + row;                     // the host keeps T below 2^31
            const bool t_ok = t < (int)p.T;
            const int tt = t_ok ? t : 0;
            const int n = tt / (int)ohw;
            const int pix = tt - n * (int)ohw;
            const int oh = pix / p.OW, ow = pix - oh * p.OW;
            const int ih0 = oh * p.stride - p.pad, iw0 = ow * p.stride - p.pad;
            // which kernel rows / columns fall inside the image for this position
            rows_in = 0;
            cols_in = 0;
            for (int a = 0; a < p.k; ++a) {
                if (t_ok && ih0 + a * p.dil >= 0 && ih0 + a * p.dil < p.H) rows_in |= 1u << a;
                if (iw0 + a * p.dil >= 0 && iw0 + a * p.dil < p.W) cols_in |= 1u << a;
            }
            base = p.x + (size_t)n * p.Cin * plane + (ptrdiff_t)ih0 * p.W + iw0;
        };
        if (n_steps > 0) decode_item();
        const int step_b = p.dil, step_a = p.dil * p.W - p.k * p.dil, step_c = (p.H - p.k * p.dil) * p.W;
        // gathers the 16 patch elements of this lane for the cursor's step (zeros outside the image, beyond the
        // patch, beyond T) and advances the cursor
        const int cblocks = p.Cin / kKBlock;                    // tap-major: channel blocks per tap
        auto gather = [&](long long, float (&v)[16]) {
            if (p.tap_major) {
                // one tap, 16 consecutive channels of this lane's position: one bounds test, loads one plane apart
                const int tap = cur_kb / cblocks, cb = cur_kb - tap * cblocks;
                const int a = tap / p.k, b = tap - a * p.k;
                const bool ok = ((rows_in >> a) & 1u) && ((cols_in >> b) & 1u);
                const float* src = base + ((size_t)(cb * kKBlock + piece0 * 4) * p.H + a * p.dil) * p.W + b * p.dil;
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = ok ? __ldg(src + (size_t)e * plane) : 0.0f;
                if (++cur_kb == p.k_blocks) {
                    cur_kb = 0;
                    cur_item += gridDim.x;
                    if (cur_item < p.n_items) decode_item();
                }
                return;
            }
            int kk = cur_kb * kKBlock + piece0 * 4;
            int ci = kk / k2;
            int r = kk - ci * k2;
            int a = r / p.k, b = r - a * p.k;
            int off = (ci * p.H + a * p.dil) * p.W + b * p.dil;      // element offset of (ci, a, b) from `base`
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const bool ok = ci < p.Cin && ((rows_in >> a) & 1u) && ((cols_in >> b) & 1u);
                v[e] = ok ? __ldg(base + off) : 0.0f;
                off += step_b;
                if (++b == p.k) {
                    b = 0;
                    off += step_a;
                    if (++a == p.k) {
                        a = 0;
                        off += step_c;
                        ++ci;
                    }
                }
            }
            if (++cur_kb == p.k_blocks) {
                cur_kb = 0;
                cur_item += gridDim.x;
                if (cur_item < p.n_items) decode_item();
            }
        };
        if (n_steps > 0) gather(0, va);
        if (n_steps > 1) gather(1, vb);
        for (long long s = 0; s < n_steps; ++s) {
            float4 w4[4];
            if ((s & 1) == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    w4[j] = make_float4(round_tf32(va[4 * j]), round_tf32(va[4 * j + 1]), round_tf32(va[4 * j + 2]), round_tf32(va[4 * j + 3]));
                if (s + 2 < n_steps) gather(s + 2, va);     // in flight during this step and the next
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    w4[j] = make_float4(round_tf32(vb[4 * j]), round_tf32(vb[4 * j + 1]), round_tf32(vb[4 * j + 2]), round_tf32(vb[4 * j + 3]));
                if (s + 2 < n_steps) gather(s + 2, vb);
            }
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_relaxed(ptx::smem_u32(&empty_bar[stage]), phase ^ 1u, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrProducerWait);
                    *abortp = 1;
                }
                break;
            }
            uint8_t* const arow = generic_base + stage * stage_bytes + row * 128;
#pragma unroll
            for (int j = 0; j < 4; ++j) *reinterpret_cast<float4*>(arow + (((piece0 + j) ^ (row & 7)) << 4)) = w4[j];
            fence_proxy_async_smem();                      // the tensor core reads these through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&full_bar[stage]));
            if (++stage == (uint32_t)p.stages) {
                stage = 0;
                phase ^= 1u;
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
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// U[co][kk'] = round_tf32(w[co][ci][a][b]) with kk' = (a * k + b) * Cin + ci (tap-major) for the producers' fast path
__global__ void implicit_weights_tap_major_kernel(const float* __restrict__ w, float* __restrict__ U, int Cout, int Cin, int k2)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long Kd = (long long)Cin * k2;
    if (gid >= (long long)Cout * Kd) return;
    const int kk = (int)(gid % Kd), co = (int)(gid / Kd);
    const int tap = kk / Cin, ci = kk - tap * Cin;
    U[gid] = round_tf32(w[((size_t)co * Cin + ci) * k2 + tap]);
}

}  // namespace

bool implicit_gemm_tap_major(int Cin) { return Cin % kKBlock == 0; }

cudaError_t launch_implicit_weights(const float* w, void* U, int Cout, int Cin, int k, int k_pad, cudaStream_t stream)
{
    if (!implicit_gemm_tap_major(Cin)) return launch_weight_round(w, U, nullptr, Cout, Cin * k * k, k_pad, STORE_TF32, stream);
    const long long total = (long long)Cout * Cin * k * k;
    implicit_weights_tap_major_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(w, static_cast<float*>(U), Cout, Cin, k * k);
    return cudaGetLastError();
}

cudaError_t implicit_gemm_setup(ImplicitGemm* ig, const GatherGeom& g, int Cout, void* U, const char** why)
{
    ig->ready = false;
    ig->Cout = Cout;
    ig->k_pad = g.k_pad;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&ig->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const long long T = (long long)g.N * g.OH * g.OW;
    contract_tiling((T + kTileM - 1) / kTileM, 1, Cout, ig->num_sms, &ig->bn, &ig->n_co_blocks);
    ig->k_blocks = (g.k_pad + kKBlock - 1) / kKBlock;
    const int stage_bytes = kABytes + ig->bn * 128;
    int stages = (kSmemBudget - 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) {
        *why = "shared memory cannot hold two pipeline stages";
        return cudaErrorInvalidValue;
    }
    ig->stages = stages;
    ig->smem_bytes = kSmemBudget;            // the full budget: at most one CTA per SM, so tensor memory is never contended
    int cols = 32;
    while (cols < 2 * ig->bn) cols *= 2;
    ig->tmem_cols = cols;
    if ((reinterpret_cast<uintptr_t>(U) & 15u) != 0 ||
        !encode_operand_map(&ig->map_u, U, 4, g.k_pad, Cout, 1, (long long)Cout * g.k_pad, ig->bn)) {
        *why = "cuTensorMapEncodeTiled failed or is unavailable";
        return cudaErrorInvalidValue;
    }
    e = cudaFuncSetAttribute(implicit_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return e;
    ig->ready = true;
    return cudaSuccess;
}

cudaError_t launch_implicit_gemm(const ImplicitGemm& ig, const float* x, const float* bias, float* y, const GatherGeom& g,
                                 int relu, int* status, cudaStream_t stream)
{
    if (!ig.ready || g.k_pad != ig.k_pad) return cudaErrorInvalidValue;
    IgParams p;
    p.x = x; p.bias = bias; p.y = y;
    p.N = g.N; p.Cin = g.Cin; p.H = g.H; p.W = g.W; p.OH = g.OH; p.OW = g.OW; p.k = g.k; p.stride = g.stride; p.pad = g.pad;
    p.dil = g.dil; p.Cout = ig.Cout;
    p.Kd = g.Cin * g.k * g.k;
    p.T = (long long)g.N * g.OH * g.OW;
    if (p.T <= 0) return cudaSuccess;
    const long long tile_blocks = (p.T + kTileM - 1) / kTileM;
    if (p.T >= (1ll << 31) - kTileM || (long long)g.Cin * g.H * g.W >= (1ll << 31)) return cudaErrorInvalidValue;
    p.n_tile_blocks = (int)tile_blocks;
    p.n_co_blocks = ig.n_co_blocks;
    p.bn = ig.bn;
    p.k_blocks = ig.k_blocks;
    p.stages = ig.stages;
    p.tmem_cols = ig.tmem_cols;
    p.n_items = tile_blocks * ig.n_co_blocks;
    p.relu = relu;
    p.tap_major = implicit_gemm_tap_major(g.Cin) ? 1 : 0;
    p.status = status;
    const long long grid = p.n_items < ig.num_sms ? p.n_items : ig.num_sms;
    return launch_overlapped(implicit_gemm_kernel, dim3((unsigned)grid), dim3(kThreads), (size_t)ig.smem_bytes, stream, ig.map_u, p);
}

}  // namespace mnnb
