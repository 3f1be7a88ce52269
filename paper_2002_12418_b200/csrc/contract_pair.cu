// The batched channel contraction of the Winograd path (Section 3.3.1 (2): the Hadamard product of Eq. 6 summed
// over channels, one matrix product per transform position) on PAIRS of SMs:
//     out[xi][co][t] = sum_c U[xi][co][c] * V[xi][t][c]
// Two CTAs of a cluster work on one 256 (tiles) x 256 (output channels) block per work item with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of V and HALF of the U tile (128 of the 256 output
// channels), the tensor cores of both SMs read both halves, and each CTA's tensor memory receives the 128 x 256
// accumulator of its own rows.  Per output a CTA therefore pulls 2 x 128 operand rows per K block from L2
// instead of 128 + 256: two thirds of the single-CTA kernel's traffic, which is what bounds that kernel (its
// shared memory holds 4 stages x 48 KB against a round trip of about 3 us; here 6 stages x 32 KB, or 3 x 64 KB
// with 128-byte rows on long K loops).
//
// Roles per CTA as in contract_umma.cu (warp 0 lane 0: TMA producer, warp 1: tensor memory and, in the cluster's
// first CTA only, the MMA issue, warps 2-5: epilogue).  Barriers: the "operands landed" barriers that count
// live in the first CTA and receive the bytes of BOTH CTAs' copies (the copies name that barrier through its
// cluster address); "stage free" and "accumulator complete" are signalled in both CTAs by one multicast
// tcgen05.commit; "accumulator drained" lives in the first CTA and collects the epilogue warps of both.  No copy
// is multicast: every CTA fetches what it stages.  All waits are local and bounded as in umma.cuh; a CTA leaves
// only after a cluster barrier, so that nothing is signalled into shared memory that is gone.
#include <cuda_bf16.h>

#include "contract_pair.h"
#include "contract_umma.h"
#include "kernels.h"
#include "umma.cuh"

namespace mnnb {

namespace {

constexpr int kPairThreads = 192;
constexpr int kRows = 128;             // rows of V, and rows of U, per CTA and stage
constexpr int kPairMaxN = 256;         // output channels per work item (MMA N): PairParams::bn, a multiple of 32
constexpr int kPairMaxStages = 8;
constexpr int kPairSmemBudget = 200 * 1024;
constexpr int kErrPairProducer = 41, kErrPairMmaFull = 42, kErrPairMmaTmem = 43, kErrPairEpilogue = 44;   // status codes

struct PairParams {
    int alpha2, n_row_blocks, n_co_blocks, k_blocks, passes, stages, Cout, merged;
    int bn;            // output channels per work item; each CTA stages bn / 2 rows of U
    long long tiles, n_items;
    float* M;
    long long m_row_stride;
    int* status;
};

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Cluster address of the shared-memory location `addr` (an address of this CTA) in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Tiled copies into THIS CTA's shared memory whose bytes are counted on a barrier given by its cluster address
// (the pair's first CTA's).
__device__ __forceinline__ void pair_load_3d(uint32_t dst_smem, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void pair_load_4d(uint32_t dst_smem, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1, int c2,
                                             int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void pair_tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void pair_tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void pair_tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (both CTAs' tensor memory) += A (128 rows from each CTA) x B (128 of the N rows from each CTA).
template <int KIND>
__device__ __forceinline__ void pair_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    const uint32_t z = 0;
    if (KIND == 0) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t"
            "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z)
            : "memory");
    } else {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t"
            "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z)
            : "memory");
    }
}
// Arrive on the barrier at this shared-memory offset in both CTAs once the MMAs issued so far have completed.
__device__ __forceinline__ void pair_commit(uint32_t bar)
{
    const unsigned short both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(both)
                 : "memory");
}

template <int SW>
__device__ __forceinline__ uint64_t pair_desc_k(uint32_t smem_addr)
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

template <int KIND, int SW>
__global__ void __launch_bounds__(kPairThreads, 1)
contract_pair_kernel(const __grid_constant__ CUtensorMap map_v_hi, const __grid_constant__ CUtensorMap map_v_lo,
                     const __grid_constant__ CUtensorMap map_u_hi, const __grid_constant__ CUtensorMap map_u_lo, PairParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kPairMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kPairMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const long long pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t tile_bytes = kRows * SW;
    const uint32_t split = p.passes == 3 ? 2u : 1u;
    const uint32_t b_bytes = (uint32_t)(p.bn / 2) * SW;              // this CTA's half of the U tile
    const uint32_t stage_bytes = (tile_bytes + b_bytes) * split;     // [A_hi][A_lo?][B_hi][B_lo?]
    const uint32_t off_a_lo = tile_bytes, off_b_hi = tile_bytes * split, off_b_lo = tile_bytes * split + b_bytes;
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_u32(&tfull_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&tempty_bar[s]), 8);      // the four epilogue warps of each CTA
        }
        abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_v_hi);
        ptx::prefetch_tensormap(&map_u_hi);
    }
    if (warp == 1) {
        pair_tmem_alloc(ptx::smem_u32(&tmem_slot), 512);
        pair_tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();                  // both CTAs' barriers exist before anything is signalled across
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    const int k_elems = (KIND == 0 ? 32 : 64) * SW / 128;   // elements of K per shared-memory row

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long item = pair; item < p.n_items && ok; item += n_pairs) {
                const int rb = (int)(item % p.n_row_blocks);
                const long long r = item / p.n_row_blocks;
                const int nb = (int)(r % p.n_co_blocks);
                const int xi = (int)(r / p.n_co_blocks);
                const int v_row = (rb * 2 + (int)rank) * kRows, u_row = nb * p.bn + (int)rank * (p.bn / 2);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&empty_bar[stage]), phase ^ 1u, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrPairProducer);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    // the first CTA's barrier counts the bytes of both CTAs' copies
                    if (rank == 0) ptx::mbar_expect_tx(ptx::smem_u32(&full_bar[stage]), 2u * stage_bytes);
                    const uint32_t bar = map_to_rank(ptx::smem_u32(&full_bar[stage]), 0);
                    const uint32_t sbase = smem_base + stage * stage_bytes;
                    if (p.merged) {
                        pair_load_4d(sbase, &map_v_hi, bar, kb * k_elems, v_row, 0, xi);
                        pair_load_4d(sbase + off_b_hi, &map_u_hi, bar, kb * k_elems, u_row, 0, xi);
                    } else {
                        pair_load_3d(sbase, &map_v_hi, bar, kb * k_elems, v_row, xi);
                        pair_load_3d(sbase + off_b_hi, &map_u_hi, bar, kb * k_elems, u_row, xi);
                        if (split == 2) {
                            pair_load_3d(sbase + off_a_lo, &map_v_lo, bar, kb * k_elems, v_row, xi);
                            pair_load_3d(sbase + off_b_lo, &map_u_lo, bar, kb * k_elems, u_row, xi);
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
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = ptx::mma_idesc(KIND == 0 ? 2 : 1, 2 * kRows, p.bn);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long item = pair; item < p.n_items && ok; item += n_pairs) {
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, abortp)) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrPairMmaTmem);
                    *abortp = 1;
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)kPairMaxN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&full_bar[stage]), phase, abortp)) {
                        if (!*abortp) atomicCAS(p.status, 0, kErrPairMmaFull);
                        *abortp = 1;
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t sbase = smem_base + stage * stage_bytes;
#pragma unroll
                    for (int ks = 0; ks < SW / 32; ++ks) {
                        const uint64_t a_hi = pair_desc_k<SW>(sbase + ks * 32);
                        const uint64_t b_hi = pair_desc_k<SW>(sbase + off_b_hi + ks * 32);
                        pair_mma<KIND>(d_tmem, a_hi, b_hi, idesc, (kb | ks) != 0 ? 1u : 0u);
                        if (split == 2) {
                            const uint64_t a_lo = pair_desc_k<SW>(sbase + off_a_lo + ks * 32);
                            const uint64_t b_lo = pair_desc_k<SW>(sbase + off_b_lo + ks * 32);
                            pair_mma<KIND>(d_tmem, a_lo, b_hi, idesc, 1u);
                            pair_mma<KIND>(d_tmem, a_hi, b_lo, idesc, 1u);
                        }
                    }
                    pair_commit(ptx::smem_u32(&empty_bar[stage]));         // the stage is free in both CTAs
                    if (++stage == (uint32_t)p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                pair_commit(ptx::smem_u32(&tfull_bar[acc]));               // accumulator complete, both CTAs
                acc ^= 1u;
                if (acc == 0) acc_phase ^= 1u;
            }
        }
    } else {
        const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (long long item = pair; item < p.n_items && ok; item += n_pairs) {
            const int rb = (int)(item % p.n_row_blocks);
            const long long r = item / p.n_row_blocks;
            const int nb = (int)(r % p.n_co_blocks);
            const int xi = (int)(r / p.n_co_blocks);
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait_bounded(ptx::smem_u32(&tfull_bar[acc]), acc_phase, abortp) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                if (lane == 0) {
                    if (!*abortp) atomicCAS(p.status, 0, kErrPairEpilogue);
                    *abortp = 1;
                }
                ok = false;
                break;
            }
            ptx::tc_fence_after();
            const long long t = ((long long)rb * 2 + rank) * kRows + q * 32 + lane;     // this thread's tile
            const bool t_ok = t < p.tiles;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * (uint32_t)kPairMaxN;
            const int co0 = nb * p.bn;
            const int n_co = min(p.bn, p.Cout - co0);
            float* dst = p.M + ((size_t)xi * p.Cout + co0) * p.m_row_stride + (t_ok ? t : 0);
            const int n_chunks = (n_co + 15) >> 4;
            uint32_t va[16], vb[16];
            auto store_chunk = [&](const uint32_t (&v)[16], int ch) {
                if (!t_ok) return;
                const int n = min(16, n_co - ch * 16);
                float* pj = dst;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < n) *pj = __uint_as_float(v[j]);
                    pj += p.m_row_stride;
                }
            };
            ptx::tmem_ld16(taddr, va);
            for (int ch = 0; ch < n_chunks; ch += 2) {
                ptx::tmem_ld_wait();
                if (ch + 1 < n_chunks) ptx::tmem_ld16(taddr + (uint32_t)((ch + 1) * 16), vb);
                store_chunk(va, ch);
                dst += 16 * p.m_row_stride;
                if (ch + 1 < n_chunks) {
                    ptx::tmem_ld_wait();
                    if (ch + 2 < n_chunks) ptx::tmem_ld16(taddr + (uint32_t)((ch + 2) * 16), va);
                    store_chunk(vb, ch + 1);
                    dst += 16 * p.m_row_stride;
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) remote_arrive(map_to_rank(ptx::smem_u32(&tempty_bar[acc]), 0));
            acc ^= 1u;
            if (acc == 0) acc_phase ^= 1u;
        }
    }

    // Teardown.  After an aborted run give copies still in flight time to land; nobody leaves before both CTAs
    // are here.
    if (*abortp) __nanosleep(200000);
    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after();
        pair_tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

cudaError_t pair_contract_setup(PairContract* pc, int mode, int alpha2, int Cout, int cin_pad, long long tiles_capacity, void* U_hi,
                                void* U_lo, void* V_hi, void* V_lo, const char** why)
{
    pc->ready = false;
    if (mode == STORE_FP32 || alpha2 < 2) {
        *why = "the pair contraction needs TF32 or BF16 operands and more than one transform position";
        return cudaErrorInvalidValue;
    }
    const int eb = store_elem_bytes(mode);
    pc->kind = eb == 2 ? 1 : 0;
    pc->passes = store_is_split(mode) ? 3 : 1;
    pc->alpha2 = alpha2;
    pc->Cout = Cout;
    pc->cin_pad = cin_pad;
    pc->tiles_capacity = tiles_capacity;
    if (((long long)cin_pad * eb) % 16 != 0) {
        *why = "operand rows must be a multiple of 16 bytes";
        return cudaErrorInvalidValue;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&pc->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (pc->num_sms < 2) {
        *why = "the pair contraction needs two SMs";
        return cudaErrorInvalidValue;
    }
    const int split = pc->passes == 3 ? 2 : 1;
    // rows of 128 bytes; 64-byte rows (twice the stages for the same bytes in flight) where 128-byte rows leave
    // fewer than four stages and the K loop is between 4 and 8 such rows long (measured: 256 channels BF16 hi + lo
    // 0.174 -> 0.172 ms with 64-byte rows, 512 channels 0.553 -> 0.525 ms with 128-byte rows)
    int sw = 128;
    pc->bn = Cout >= kPairMaxN ? kPairMaxN : (Cout + 31) / 32 * 32;
    if ((kPairSmemBudget - 1024) / ((kRows + pc->bn / 2) * sw * split) < 4 && cin_pad * eb >= 4 * 64 && cin_pad * eb < 8 * 128) sw = 64;
    pc->sw = sw;
    const int k_elems = sw / eb;
    pc->k_blocks = (cin_pad + k_elems - 1) / k_elems;
    int stages = (kPairSmemBudget - 1024) / ((kRows + pc->bn / 2) * sw * split);
    if (stages > kPairMaxStages) stages = kPairMaxStages;
    if (stages < 2) {
        *why = "shared memory cannot hold two pipeline stages";
        return cudaErrorInvalidValue;
    }
    pc->stages = stages;
    pc->smem_bytes = kPairSmemBudget;
    const long long u_plane = (long long)Cout * cin_pad, v_plane = tiles_capacity * cin_pad;
    pc->merged = 0;
    bool ok = true;
    if (split == 2) {
        const long long dv = static_cast<char*>(V_lo) - static_cast<char*>(V_hi), du = static_cast<char*>(U_lo) - static_cast<char*>(U_hi);
        if (encode_operand_pair_map(&pc->map_v_hi, V_hi, dv, eb, cin_pad, tiles_capacity, alpha2, v_plane, kRows, sw) &&
            encode_operand_pair_map(&pc->map_u_hi, U_hi, du, eb, cin_pad, Cout, alpha2, u_plane, pc->bn / 2, sw)) {
            pc->merged = 1;
            pc->map_v_lo = pc->map_v_hi;
            pc->map_u_lo = pc->map_u_hi;
        }
    }
    if (!pc->merged) {
        ok = encode_operand_map_sw(&pc->map_v_hi, V_hi, eb, cin_pad, tiles_capacity, alpha2, v_plane, kRows, sw) &&
             encode_operand_map_sw(&pc->map_u_hi, U_hi, eb, cin_pad, Cout, alpha2, u_plane, pc->bn / 2, sw);
        if (ok && split == 2)
            ok = encode_operand_map_sw(&pc->map_v_lo, V_lo, eb, cin_pad, tiles_capacity, alpha2, v_plane, kRows, sw) &&
                 encode_operand_map_sw(&pc->map_u_lo, U_lo, eb, cin_pad, Cout, alpha2, u_plane, pc->bn / 2, sw);
        if (ok && split == 1) {
            pc->map_v_lo = pc->map_v_hi;
            pc->map_u_lo = pc->map_u_hi;
        }
    }
    if (!ok) {
        *why = "cuTensorMapEncodeTiled failed or is unavailable";
        return cudaErrorInvalidValue;
    }
    for (auto kern : {contract_pair_kernel<0, 128>, contract_pair_kernel<1, 128>, contract_pair_kernel<0, 64>,
                      contract_pair_kernel<1, 64>}) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBudget);
        if (e != cudaSuccess) return e;
    }
    pc->ready = true;
    return cudaSuccess;
}

cudaError_t launch_contract_pair(const PairContract& pc, long long tiles, float* M, long long m_row_stride, int* status,
                                 cudaStream_t stream)
{
    if (!pc.ready) return cudaErrorInvalidValue;
    if (tiles <= 0) return cudaSuccess;
    if (tiles > pc.tiles_capacity) return cudaErrorInvalidValue;
    PairParams p;
    p.alpha2 = pc.alpha2;
    p.n_row_blocks = (int)((tiles + 2 * kRows - 1) / (2 * kRows));
    p.bn = pc.bn;
    p.n_co_blocks = (pc.Cout + pc.bn - 1) / pc.bn;
    p.k_blocks = pc.k_blocks;
    p.passes = pc.passes;
    p.stages = pc.stages;
    p.Cout = pc.Cout;
    p.merged = pc.merged;
    p.tiles = tiles;
    p.n_items = (long long)p.n_row_blocks * p.n_co_blocks * pc.alpha2;
    p.M = M;
    p.m_row_stride = m_row_stride;
    p.status = status;
    const long long max_pairs = pc.num_sms / 2;
    const long long pairs = p.n_items < max_pairs ? p.n_items : max_pairs;
    auto kern = pc.kind == 0 ? (pc.sw == 64 ? contract_pair_kernel<0, 64> : contract_pair_kernel<0, 128>)
                             : (pc.sw == 64 ? contract_pair_kernel<1, 64> : contract_pair_kernel<1, 128>);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = (size_t)pc.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, pc.map_v_hi, pc.map_v_lo, pc.map_u_hi, pc.map_u_lo, p);
}

}  // namespace mnnb
