// Winograd input transform V = B^T d B (Eq. 6) as a persistent, warp-specialised kernel.
//
// Work item = (image, tile row, segment of up to `txs` tiles of that row, block of 64
// channels).  The alpha input rows of an item are staged in a ring of shared-memory
// buffers laid out [row][channel slot][column]; the number of staged columns `wb` is an
// odd multiple of 4 words, so that 32 lanes reading 128-bit vectors from 32 consecutive
// slots touch every bank once.  When the image rows are 16-byte aligned (W a multiple of
// 4) one loader warp issues TMA box copies, one per input row (box = 64 channels x wb
// columns; or two boxes of 32 channels, even and odd, through a 5-D view of x that splits
// the channel parity); everything outside the image, including the zero padding of the
// convolution and channels beyond Cin, arrives as zeros, so several items are in flight
// with no load instructions at all.  Otherwise eight loader warps issue contiguous cp.async
// copies with explicit zero fill.  The remaining warps take (item, tile) units in order.  A
// lane transforms one tile of TWO adjacent channels held as packed fp32 pairs (packed
// fp32x2 multiply-adds), or of one channel for alpha >= 8 where a pair would not fit the
// register file, and writes one 128- or 256-byte row piece of V[xi][tile][channel] per
// warp store.
//
// When the interpolation points are symmetric (0, +-p1, +-p2, ..., infinity; alpha even)
// B^T has a fixed zero pattern and its +p / -p rows share coefficients up to sign
// (the generator polynomial of Eq. 8 is odd), so each 1-D pass needs about half the
// multiplies of the dense form.  The host checks the pattern on the generated matrix
// and otherwise selects the dense form.
//
// Loader and compute warps hand buffers over through mbarriers; every wait is bounded
// and reports through the plan's status word instead of hanging.
#pragma once
#include <cuda_bf16.h>

#include <cstring>
#include <type_traits>

#include "kernels.h"
#include "umma.cuh"

namespace mnnb {
namespace wino {

constexpr int kItChannels = 64;         // channels per work item
constexpr int kItWarps = 16;
constexpr int kItThreads = 32 * kItWarps;
constexpr int kItMaxBuffers = 6;
constexpr int kItCopySlots = 12;        // cp.async path: at most 32 * 12 copies per channel of an item
constexpr int kItSmemBudget = 200 * 1024;
constexpr int kErrInputLoaderWait = 11, kErrInputComputeWait = 12;

struct MatBt2 { float2 v[12 * 12]; };   // B^T with every entry duplicated into a pair

struct InputItems {
    int txs;            // tiles per item
    int nseg;           // segments per tile row
    int wb;             // staged columns per channel row: 4 x odd words
    int nbuf;           // ring depth
    int cblocks;        // blocks of 64 channels
    int use_tma;        // 1: TMA box copies (W % 4 == 0), 0: cp.async
    int vec;            // alignment of the staged column grid in elements: 4 with TMA, else 2 or 1
    int loader_warps;   // 1 with TMA, else 8
    int buf_words;      // words per buffer = alpha * 64 * wb
    long long n_items;
};

__device__ __forceinline__ float round_tf32_v(float v)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

// ---- value types: one channel (float) or two adjacent channels (float2) per lane ----
__device__ __forceinline__ float v_mul(float2 c, float a) { return c.x * a; }
__device__ __forceinline__ float v_fma(float2 c, float a, float acc) { return fmaf(c.x, a, acc); }
__device__ __forceinline__ float v_add(float a, float b) { return a + b; }
__device__ __forceinline__ float v_sub(float a, float b) { return a - b; }
__device__ __forceinline__ float2 v_mul(float2 c, float2 a) { return __fmul2_rn(c, a); }
__device__ __forceinline__ float2 v_fma(float2 c, float2 a, float2 acc) { return __ffma2_rn(c, a, acc); }
__device__ __forceinline__ float2 v_add(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 v_sub(float2 a, float2 b) { return __ffma2_rn(make_float2(-1.0f, -1.0f), b, a); }
__device__ __forceinline__ float v_make(float a, float, float) { return a; }
__device__ __forceinline__ float2 v_make(float a, float b, float2) { return make_float2(a, b); }

// One 1-D pass o = B^T d, outputs LO .. HI - 1 only (the others are left untouched).  SYM: the
// symmetric-point structure described above; LO and HI are then 0 / ALPHA or odd, so that a +p / -p pair of
// rows is never cut.
template <int ALPHA, bool SYM, typename T, int LO = 0, int HI = ALPHA>
__device__ __forceinline__ void pass_1d(const T (&d)[ALPHA], T (&o)[ALPHA], const MatBt2& Bt)
{
    if (SYM) {
        static_assert((LO == 0 || (LO & 1)) && (HI == ALPHA || (HI & 1)), "a pass may not cut a +p / -p pair");
        if (LO == 0) {
            // row of the point 0: even powers only
            T s = v_mul(Bt.v[0], d[0]);
#pragma unroll
            for (int r = 2; r < ALPHA; r += 2) s = v_fma(Bt.v[r], d[r], s);
            o[0] = s;
        }
        if (HI == ALPHA) {
            // row of the point at infinity: odd powers only
            T s = v_mul(Bt.v[(ALPHA - 1) * ALPHA + 1], d[1]);
#pragma unroll
            for (int r = 3; r < ALPHA; r += 2) s = v_fma(Bt.v[(ALPHA - 1) * ALPHA + r], d[r], s);
            o[ALPHA - 1] = s;
        }
        // +p / -p pairs: even part E (r = 2, 4, ..), odd part O (r = 1, 3, ..); rows are E + O and E - O
#pragma unroll
        for (int p = 1; p < ALPHA - 1; p += 2) {
            if (p < LO || p + 1 >= HI) continue;
            T e = v_mul(Bt.v[p * ALPHA + 2], d[2]);
#pragma unroll
            for (int r = 4; r < ALPHA - 1; r += 2) e = v_fma(Bt.v[p * ALPHA + r], d[r], e);
            T od = v_mul(Bt.v[p * ALPHA + 1], d[1]);
#pragma unroll
            for (int r = 3; r < ALPHA - 1; r += 2) od = v_fma(Bt.v[p * ALPHA + r], d[r], od);
            o[p] = v_add(e, od);
            o[p + 1] = v_sub(e, od);
        }
    } else {
#pragma unroll
        for (int i = LO; i < HI; ++i) {
            T s = v_mul(Bt.v[i * ALPHA], d[0]);
#pragma unroll
            for (int r = 1; r < ALPHA; ++r) s = v_fma(Bt.v[i * ALPHA + r], d[r], s);
            o[i] = s;
        }
    }
}

// ---- stores in the operand formats (lane's channel, or channel pair, at byte pointers hi / lo) ----
template <int MODE>
__device__ __forceinline__ void put(char* hi, char* lo, float v)
{
    if (MODE == STORE_TF32) {
        *reinterpret_cast<float*>(hi) = round_tf32_v(v);
    } else if (MODE == STORE_BF16) {
        *reinterpret_cast<__nv_bfloat16*>(hi) = __float2bfloat16_rn(v);
    } else if (MODE == STORE_TF32_SPLIT) {
        const float h = round_tf32_v(v);
        *reinterpret_cast<float*>(hi) = h;
        *reinterpret_cast<float*>(lo) = round_tf32_v(v - h);
    } else if (MODE == STORE_BF16_SPLIT) {
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        *reinterpret_cast<__nv_bfloat16*>(hi) = h;
        *reinterpret_cast<__nv_bfloat16*>(lo) = __float2bfloat16_rn(v - __bfloat162float(h));
    } else {
        *reinterpret_cast<float*>(hi) = v;
    }
}
template <int MODE>
__device__ __forceinline__ void put(char* hi, char* lo, float2 v)
{
    if (MODE == STORE_TF32) {
        *reinterpret_cast<float2*>(hi) = make_float2(round_tf32_v(v.x), round_tf32_v(v.y));
    } else if (MODE == STORE_BF16) {
        *reinterpret_cast<__nv_bfloat162*>(hi) = __floats2bfloat162_rn(v.x, v.y);
    } else if (MODE == STORE_TF32_SPLIT) {
        const float2 h = make_float2(round_tf32_v(v.x), round_tf32_v(v.y));
        *reinterpret_cast<float2*>(hi) = h;
        const float2 l = v_sub(v, h);
        *reinterpret_cast<float2*>(lo) = make_float2(round_tf32_v(l.x), round_tf32_v(l.y));
    } else if (MODE == STORE_BF16_SPLIT) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(v.x, v.y);
        const float2 l = v_sub(v, __bfloat1622float2(h));
        *reinterpret_cast<__nv_bfloat162*>(hi) = h;
        *reinterpret_cast<__nv_bfloat162*>(lo) = __floats2bfloat162_rn(l.x, l.y);
    } else {
        *reinterpret_cast<float2*>(hi) = v;
    }
}

// Row pass of one tile: h[r][j'] = sum_j d[r][j] Bt[j'][j].  p0 (and p1 for the second channel of a pair)
// point at the 16-byte aligned vector of staged row 0 that holds the tile's first column; OFF = that
// column's index in the vector; row_words = words between staged rows.  Only the columns LO .. HI - 1 of h are
// computed.
template <int ALPHA, bool SYM, int OFF, typename T, int LO = 0, int HI = ALPHA>
__device__ __forceinline__ void rows_pass(const float* p0, const float* p1, int row_words, const MatBt2& Bt,
                                          T (&h)[ALPHA][ALPHA])
{
    constexpr int NV = (OFF + ALPHA + 3) / 4;
    constexpr bool kPair = std::is_same<T, float2>::value;
#pragma unroll
    for (int r = 0; r < ALPHA; ++r) {
        float a[4 * NV], b[4 * NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float4 q = *reinterpret_cast<const float4*>(p0 + r * row_words + 4 * v);
            a[4 * v] = q.x; a[4 * v + 1] = q.y; a[4 * v + 2] = q.z; a[4 * v + 3] = q.w;
            if (kPair) {
                const float4 s = *reinterpret_cast<const float4*>(p1 + r * row_words + 4 * v);
                b[4 * v] = s.x; b[4 * v + 1] = s.y; b[4 * v + 2] = s.z; b[4 * v + 3] = s.w;
            } else {
                b[4 * v] = b[4 * v + 1] = b[4 * v + 2] = b[4 * v + 3] = 0.0f;
            }
        }
        T d[ALPHA];
#pragma unroll
        for (int j = 0; j < ALPHA; ++j) d[j] = v_make(a[OFF + j], b[OFF + j], T());
        pass_1d<ALPHA, SYM, T, LO, HI>(d, h[r], Bt);
        // large tiles: keep the compiler from hoisting the loads of all rows above the arithmetic of the first,
        // which would cost more registers than the intermediate itself
        if (ALPHA >= 8) asm volatile("" ::: "memory");
    }
}

// Column pass and stores: V[i][j] = sum_r Bt[i][r] h[r][j], transform position xi = i * alpha + j, for the
// columns j = LO .. HI - 1 (hi / lo point at position (0, 0)).
template <int ALPHA, bool SYM, int MODE, typename T, int LO = 0, int HI = ALPHA>
__device__ __forceinline__ void cols_pass_store(const T (&h)[ALPHA][ALPHA], const MatBt2& Bt, char* hi, char* lo,
                                                long long plane_bytes)
{
    const long long row_step = plane_bytes * ALPHA;   // from transform position (i, j) to (i + 1, j)
    hi += plane_bytes * LO;
    lo += plane_bytes * LO;
#pragma unroll
    for (int j = LO; j < HI; ++j) {
        T col[ALPHA], o[ALPHA];
#pragma unroll
        for (int r = 0; r < ALPHA; ++r) col[r] = h[r][j];
        pass_1d<ALPHA, SYM, T>(col, o, Bt);
        char* ph = hi;
        char* pl = lo;
#pragma unroll
        for (int i = 0; i < ALPHA; ++i) {
            put<MODE>(ph, pl, o[i]);
            ph += row_step;
            pl += row_step;
        }
        hi += plane_bytes;
        lo += plane_bytes;
    }
}

// One tile (columns LO .. HI - 1 of its transform): row pass from the staged rows, column pass, stores.
// `off` = index of the tile's first input column in its 16-byte vector (0..3).
template <int ALPHA, bool SYM, typename T, int LO, int HI>
__device__ __forceinline__ void tile_columns(const float* p0, const float* p1, int row_words, int off, const MatBt2& Bt,
                                             int mode, char* hi, char* lo, long long plane_bytes)
{
    T h[ALPHA][ALPHA];
    switch (off) {
        case 0: rows_pass<ALPHA, SYM, 0, T, LO, HI>(p0, p1, row_words, Bt, h); break;
        case 1: rows_pass<ALPHA, SYM, 1, T, LO, HI>(p0, p1, row_words, Bt, h); break;
        case 2: rows_pass<ALPHA, SYM, 2, T, LO, HI>(p0, p1, row_words, Bt, h); break;
        default: rows_pass<ALPHA, SYM, 3, T, LO, HI>(p0, p1, row_words, Bt, h); break;
    }
    switch (mode) {
        case STORE_TF32: cols_pass_store<ALPHA, SYM, STORE_TF32, T, LO, HI>(h, Bt, hi, lo, plane_bytes); break;
        case STORE_BF16: cols_pass_store<ALPHA, SYM, STORE_BF16, T, LO, HI>(h, Bt, hi, lo, plane_bytes); break;
        case STORE_TF32_SPLIT: cols_pass_store<ALPHA, SYM, STORE_TF32_SPLIT, T, LO, HI>(h, Bt, hi, lo, plane_bytes); break;
        case STORE_BF16_SPLIT: cols_pass_store<ALPHA, SYM, STORE_BF16_SPLIT, T, LO, HI>(h, Bt, hi, lo, plane_bytes); break;
        default: cols_pass_store<ALPHA, SYM, STORE_FP32, T, LO, HI>(h, Bt, hi, lo, plane_bytes); break;
    }
}

// One tile.  Up to alpha = 6 the alpha x alpha intermediate stays in registers; from alpha = 8 on the tile is
// done in two or three sweeps of at most 5 columns each (the staged rows are read once per sweep), which keeps
// the intermediate at alpha x 5 values and the kernel clear of local-memory spills at 128 registers.
template <int ALPHA, bool SYM, typename T>
__device__ __forceinline__ void transform_tile(const float* p0, const float* p1, int row_words, int off, const MatBt2& Bt,
                                               int mode, char* hi, char* lo, long long plane_bytes)
{
    if constexpr (ALPHA < 8) {
        tile_columns<ALPHA, SYM, T, 0, ALPHA>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
    } else if constexpr (ALPHA <= 10) {
        tile_columns<ALPHA, SYM, T, 0, 5>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
        tile_columns<ALPHA, SYM, T, 5, ALPHA>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
    } else {
        tile_columns<ALPHA, SYM, T, 0, 5>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
        tile_columns<ALPHA, SYM, T, 5, 9>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
        tile_columns<ALPHA, SYM, T, 9, ALPHA>(p0, p1, row_words, off, Bt, mode, hi, lo, plane_bytes);
    }
}

// Shared-memory slot of channel c (0..63) of an item.  With channel pairs, lane l works on channels
// 2l and 2l + 1 and finds them in slots l and 32 + l, so that both reads walk consecutive slots.
template <bool PAIR>
__device__ __forceinline__ int slot_of(int c)
{
    return PAIR ? ((c & 1) * 32 + (c >> 1)) : c;
}

template <int ALPHA, bool SYM, bool PAIR>
__global__ void __launch_bounds__(kItThreads, 1)
input_transform_ws_kernel(const float* __restrict__ x, const __grid_constant__ CUtensorMap xmap, char* V_hi, char* V_lo,
                          WinoGeom g, InputItems it, int mode, const __grid_constant__ MatBt2 Bt, int* status)
{
    extern __shared__ __align__(128) float s_buf[];
    __shared__ __align__(8) uint64_t full_bar[kItMaxBuffers];
    __shared__ __align__(8) uint64_t empty_bar[kItMaxBuffers];
    __shared__ int4 item_desc[kItMaxBuffers];      // (image, tile row, first tile, channel block) of the item in each buffer
    __shared__ int abort_flag;
    volatile int* abortp = &abort_flag;
    using T = typename std::conditional<PAIR, float2, float>::type;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kHalves = PAIR ? 1 : 2;                 // units per tile: one for 64 channels, or two of 32
    const int units_per_item = it.txs * kHalves;
    const int n_compute = kItWarps - it.loader_warps;
    const int row_words = kItChannels * it.wb;            // words between staged rows
    if (threadIdx.x == 0) {
        for (int b = 0; b < it.nbuf; ++b) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[b]), it.use_tma ? 1u : 32u * (uint32_t)it.loader_warps);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[b]), (uint32_t)n_compute);
        }
        abort_flag = 0;
        ptx::fence_barrier_init();
        if (it.use_tma) ptx::prefetch_tensormap(&xmap);
    }
    __syncthreads();
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    // items of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ... (32-bit: the host keeps n_items below 2^31)
    const unsigned first = blockIdx.x, n_items = (unsigned)it.n_items;
    const unsigned n_local = first < n_items ? (n_items - first + gridDim.x - 1) / gridDim.x : 0;
    const int eb = (mode == STORE_BF16 || mode == STORE_BF16_SPLIT) ? 2 : 4;

    if (warp < it.loader_warps) {
        // ------------------------------- loaders -------------------------------
        int b = 0;
        uint32_t round = 0;
        int copy_r[kItCopySlots], copy_j[kItCopySlots];       // cp.async path: this lane's (row, first column) per step
        {
            const int per_row = it.wb / it.vec;
#pragma unroll
            for (int i = 0; i < kItCopySlots; ++i) {
                const int e = lane + 32 * i;
                const int r = e / per_row;
                copy_r[i] = (!it.use_tma && r < ALPHA) ? r : -1;
                copy_j[i] = (e - r * per_row) * it.vec;
            }
        }
        for (unsigned li = 0; li < n_local; ++li) {
            if (round > 0 && !ptx::mbar_wait_relaxed(ptx::smem_u32(&empty_bar[b]), (round - 1) & 1u, abortp)) {
                if (!*abortp && status) atomicCAS(status, 0, kErrInputLoaderWait | (int)(min(li, 0xFFFFu) << 8) | (int)((blockIdx.x & 0x7Fu) << 24));
                *abortp = 1;
                break;
            }
            unsigned item = first + li * gridDim.x;
            const int cb = (int)(item % (unsigned)it.cblocks); item /= (unsigned)it.cblocks;
            const int seg = (int)(item % (unsigned)it.nseg); item /= (unsigned)it.nseg;
            const int ty = (int)(item % (unsigned)g.th);
            const int img = (int)(item / (unsigned)g.th);
            const int tx0 = seg * it.txs;
            const int ih0 = ty * g.m - g.pad, iw0 = tx0 * g.m - g.pad;
            const int a0 = iw0 - ((iw0 % it.vec + it.vec) % it.vec);      // first staged column, on the vector grid
            const int c0 = cb * kItChannels;
            if (threadIdx.x == 0) item_desc[b] = make_int4(img, ty, tx0, cb);
            const uint32_t sbuf = ptx::smem_u32(s_buf) + (uint32_t)b * (uint32_t)it.buf_words * 4u;
            const uint32_t bar = ptx::smem_u32(&full_bar[b]);
            if (it.use_tma) {
                if (lane == 0) ptx::mbar_expect_tx(bar, (uint32_t)it.buf_words * 4u);
                __syncwarp();
                if (PAIR) {
                    // lane = (row, parity): 32 channels of one parity of one input row
                    if (lane < 2 * ALPHA) {
                        const int r = lane >> 1, par = lane & 1;
                        ptx::tma_load_5d(sbuf + (uint32_t)(r * row_words + par * 32 * it.wb) * 4u, &xmap, bar, a0, ih0 + r, par,
                                         c0 >> 1, img);
                    }
                } else {
                    if (lane < ALPHA) ptx::tma_load_4d(sbuf + (uint32_t)(lane * row_words) * 4u, &xmap, bar, a0, ih0 + lane, c0, img);
                }
            } else {
                // contiguous copies: consecutive lanes take consecutive staged elements of one channel (rows of wb
                // columns, alpha rows).  A lane's elements have the same (row, column) in every channel and item,
                // so they are decoded once (copy_r / copy_j, before the item loop).
                const float* ximg = x + (size_t)img * g.Cin * g.H * g.W;
                uint32_t nbytes[kItCopySlots];
#pragma unroll
                for (int i = 0; i < kItCopySlots; ++i) {
                    const int ih = ih0 + copy_r[i], iw = a0 + copy_j[i];
                    nbytes[i] = (copy_r[i] >= 0 && ih >= 0 && ih < g.H && iw >= 0 && iw + it.vec <= g.W) ? 4u * (uint32_t)it.vec : 0u;
                }
                for (int c = warp; c < kItChannels; c += it.loader_warps) {
                    const int ci = c0 + c;
                    const bool c_ok = ci < g.Cin;
                    const float* src = ximg + ((size_t)(c_ok ? ci : 0) * g.H + ih0) * g.W + a0;
                    const uint32_t dst = sbuf + (uint32_t)(slot_of<PAIR>(c) * it.wb) * 4u;
#pragma unroll
                    for (int i = 0; i < kItCopySlots; ++i) {
                        if (copy_r[i] < 0) break;
                        const uint32_t nb = c_ok ? nbytes[i] : 0u;
                        const uint32_t d = dst + (uint32_t)(copy_r[i] * row_words + copy_j[i]) * 4u;
                        const float* sp = nb ? src + copy_r[i] * g.W + copy_j[i] : ximg;
                        if (it.vec == 2) ptx::cp_async_8(d, sp, nb);
                        else ptx::cp_async_4(d, sp, nb);
                    }
                }
                ptx::cp_async_arrive_noinc(bar);
            }
            if (++b == it.nbuf) {
                b = 0;
                ++round;
            }
        }
        if (!it.use_tma) ptx::cp_async_wait_all();
    } else {
        // ------------------------------- compute -------------------------------
        const int cw = warp - it.loader_warps;
        const long long plane_bytes = (long long)g.v_plane * eb;
        // Every compute warp waits for every item, in order, and releases it, so that no buffer can run more
        // than one phase ahead of any warp (copies of different items may land out of order, and a parity
        // wait cannot tell a phase that is two behind from one that is done).  Of the item's units
        // (tile[, half]) a warp transforms those whose running index is congruent to it modulo n_compute.
        int b = 0, start = 0;                              // start = (li * units_per_item) mod n_compute
        uint32_t round = 0;
        for (unsigned li = 0; li < n_local; ++li) {
            if (!ptx::mbar_wait_relaxed(ptx::smem_u32(&full_bar[b]), round & 1u, abortp)) {
                if (!*abortp && status)
                    atomicCAS(status, 0, kErrInputComputeWait | (int)(min(li, 0xFFFFu) << 8) | (int)((blockIdx.x & 0x7Fu) << 24));
                *abortp = 1;
                break;
            }
            const int4 desc = item_desc[b];
            const int img = desc.x, ty = desc.y, tx0 = desc.z, cb = desc.w;
            const int iw0 = tx0 * g.m - g.pad;
            const int lead = (iw0 % it.vec + it.vec) % it.vec;             // staged columns ahead of the segment
            for (int within = (cw - start + n_compute) % n_compute; within < units_per_item; within += n_compute) {
                const int t = PAIR ? within : (within >> 1), half = PAIR ? 0 : (within & 1);
                const int tx = tx0 + t;
                const int c = cb * kItChannels + (PAIR ? 2 * lane : half * 32 + lane);
                if (tx < g.tw && c < g.cin_pad) {
                    const long long tile = ((long long)img * g.th + ty) * g.tw + tx;
                    const int s0 = lead + t * g.m;                         // staged column of the tile's first input column
                    const float* p0 = s_buf + (size_t)b * it.buf_words + (size_t)(PAIR ? lane : half * 32 + lane) * it.wb + (s0 & ~3);
                    const float* p1 = p0 + 32 * it.wb;
                    const long long off = (tile * g.cin_pad + c) * eb;
                    transform_tile<ALPHA, SYM, T>(p0, p1, row_words, s0 & 3, Bt, mode, V_hi + off, V_lo ? V_lo + off : nullptr,
                                                  plane_bytes);
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&empty_bar[b]));
            start += units_per_item % n_compute;
            if (start >= n_compute) start -= n_compute;
            if (++b == it.nbuf) {
                b = 0;
                ++round;
            }
        }
    }
    // After a wait ran out, give copies still in flight time to land before this CTA's shared memory is released.
    if (*abortp) __nanosleep(200000);
}

// Small planes whose rows are not 16-byte aligned (W not a multiple of 4: 14 x 14, 7 x 7, ...), which TMA
// cannot address row by row: one CTA per (image, block of 64 channels) copies the 64 contiguous channel planes
// into shared memory with plain coalesced loads, each plane zero-padded to hp rows x wp columns (image row ih
// at staged row ih + pad, image column iw at staged column lead + iw; everything else stays zero, which is the
// convolution's padding and the overhang of the last tiles), and then transforms ALL tiles of the image from
// there with the same row and column passes as the ring-buffer kernel: a tile's vectors are found exactly as
// there, with wp words between staged rows.  hp and wp / 4 are odd, so that 32 lanes reading 128-bit vectors
// from 32 consecutive planes touch every bank once.
struct PlaneItems {
    int hp, wp, lead, cblocks;
};

template <int ALPHA, bool SYM, bool PAIR>
__global__ void __launch_bounds__(kItThreads, 1)
input_transform_plane_kernel(const float* __restrict__ x, char* V_hi, char* V_lo, WinoGeom g, PlaneItems pi, int mode,
                             const __grid_constant__ MatBt2 Bt)
{
    extern __shared__ __align__(128) float s_buf[];
    using T = typename std::conditional<PAIR, float2, float>::type;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int plane = pi.hp * pi.wp;
    {
        float4* z = reinterpret_cast<float4*>(s_buf);
        for (int i = threadIdx.x; i < kItChannels * plane / 4; i += kItThreads) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    __syncthreads();
    const int img = blockIdx.x / pi.cblocks, cb = blockIdx.x - img * pi.cblocks;
    const int c0 = cb * kItChannels, hw = g.H * g.W;
    const float* ximg = x + (size_t)img * g.Cin * hw;
    if (hw <= 256) {
        // A lane's pixels (lane, lane + 32, ...) land at the same offsets in every plane: decode them once, then
        // copy two channels per step, sixteen loads in flight per lane.  Channels beyond Cin stay zero.
        int off[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int p = k * 32 + lane, r = p / g.W;
            off[k] = p < hw ? (g.pad + r) * pi.wp + pi.lead + (p - r * g.W) : -1;
        }
        for (int c = warp; c < kItChannels; c += 2 * kItWarps) {
            float v[2][8];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int ci = c0 + c + j * kItWarps;
                const float* src = ximg + (size_t)(ci < g.Cin ? ci : 0) * hw + lane;
#pragma unroll
                for (int k = 0; k < 8; ++k) v[j][k] = (off[k] >= 0 && ci < g.Cin) ? __ldg(src + 32 * k) : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float* dst = s_buf + (size_t)slot_of<PAIR>(c + j * kItWarps) * plane;
                if (c0 + c + j * kItWarps < g.Cin) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (off[k] >= 0) dst[off[k]] = v[j][k];
                }
            }
        }
    } else {
        // A warp copies channels warp, warp + 16, ... (kItChannels / kItWarps of them), 32 pixels per step; the
        // steps of all its channels form one sequence, taken eight at a time: eight loads in flight per lane,
        // then the eight stores.  Channels beyond Cin are skipped: their planes stay zero.
        constexpr int kChPerWarp = kItChannels / kItWarps;
        const int steps_per_ch = (hw + 31) / 32, n_steps = kChPerWarp * steps_per_ch;
        for (int s0 = 0; s0 < n_steps; s0 += 8) {
            float v[8];
            int dst[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int st = s0 + k;
                const int cw = st / steps_per_ch, p = (st - cw * steps_per_ch) * 32 + lane;
                const int c = warp + cw * kItWarps, ci = c0 + c;
                const bool ok = st < n_steps && p < hw && ci < g.Cin;
                v[k] = ok ? __ldg(ximg + (size_t)ci * hw + p) : 0.0f;
                const int r = p / g.W, col = p - r * g.W;
                dst[k] = ok ? slot_of<PAIR>(c) * plane + (g.pad + r) * pi.wp + pi.lead + col : -1;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (dst[k] >= 0) s_buf[dst[k]] = v[k];
        }
    }
    __syncthreads();
    const int eb = (mode == STORE_BF16 || mode == STORE_BF16_SPLIT) ? 2 : 4;
    const long long plane_bytes = (long long)g.v_plane * eb;
    const int units = g.th * g.tw * (PAIR ? 1 : 2);                // (tile[, half of the channel block])
    for (int u = warp; u < units; u += kItWarps) {
        const int ti = PAIR ? u : (u >> 1), half = PAIR ? 0 : (u & 1);
        const int ty = ti / g.tw, tx = ti - ty * g.tw;
        const int c = c0 + (PAIR ? 2 * lane : half * 32 + lane);
        if (c >= g.cin_pad) continue;
        const long long tile = ((long long)img * g.th + ty) * g.tw + tx;
        const int s0 = pi.lead + tx * g.m - g.pad;                 // staged column of the tile's first input column
        const float* p0 = s_buf + (size_t)(PAIR ? lane : half * 32 + lane) * plane + (size_t)(ty * g.m) * pi.wp + (s0 & ~3);
        const float* p1 = p0 + (size_t)32 * plane;
        const long long off = (tile * g.cin_pad + c) * eb;
        transform_tile<ALPHA, SYM, T>(p0, p1, pi.wp, s0 & 3, Bt, mode, V_hi + off, V_lo ? V_lo + off : nullptr, plane_bytes);
    }
}

// Padded plane shape for input_transform_plane_kernel; false when 64 planes do not fit the shared-memory budget.
inline bool plan_plane_items(const WinoGeom& g, int alpha, PlaneItems* pi, size_t* smem)
{
    const int lead = (g.pad + 3) / 4 * 4;
    int hp = (g.th - 1) * g.m + alpha;
    if (hp < g.H + g.pad) hp = g.H + g.pad;
    if ((hp & 1) == 0) ++hp;
    // columns: the image, and whole 4-wide vectors up to three columns past the last tile
    int wp = lead - g.pad + (g.tw - 1) * g.m + alpha + 3;
    if (wp < lead + g.W) wp = lead + g.W;
    wp = (wp + 3) / 4 * 4;
    if (((wp / 4) & 1) == 0) wp += 4;
    const long long bytes = (long long)kItChannels * hp * wp * 4;
    const long long blocks = (long long)g.images * ((g.cin_pad + kItChannels - 1) / kItChannels);
    if (bytes > kItSmemBudget || blocks > 2147483647ll) return false;
    pi->hp = hp;
    pi->wp = wp;
    pi->lead = lead;
    pi->cblocks = (g.cin_pad + kItChannels - 1) / kItChannels;
    *smem = (size_t)bytes;
    return true;
}

// True when Bt (alpha x alpha, row-major) has the zero pattern and the +p / -p row symmetry
// that pass_1d<.., SYM = true> assumes.
inline bool bt_has_symmetric_structure(const float* Bt, int alpha)
{
    if (alpha < 4 || (alpha & 1)) return false;
    for (int r = 0; r < alpha; ++r) {
        if ((r & 1) && Bt[r] != 0.0f) return false;                                  // point 0: even powers only
        if (!(r & 1) && Bt[(alpha - 1) * alpha + r] != 0.0f) return false;            // infinity: odd powers only
    }
    for (int p = 1; p < alpha - 1; p += 2) {
        const float* a = Bt + p * alpha;
        const float* b = Bt + (p + 1) * alpha;
        if (a[0] != 0.0f || b[0] != 0.0f || a[alpha - 1] != 0.0f || b[alpha - 1] != 0.0f) return false;
        for (int r = 1; r < alpha - 1; ++r)
            if (b[r] != ((r & 1) ? -a[r] : a[r])) return false;
    }
    return true;
}

// Item geometry.
inline bool plan_input_items(const WinoGeom& g, int alpha, bool tma_ok, int num_sms, InputItems* it)
{
    it->use_tma = tma_ok ? 1 : 0;
    it->vec = tma_ok ? 4 : ((g.W % 2 == 0) ? 2 : 1);
    it->loader_warps = tma_ok ? 1 : 8;
    it->cblocks = (g.cin_pad + kItChannels - 1) / kItChannels;
    // Candidates: the longest segment for which at least three buffers fit, and up to three finer splits;
    // the one with the shortest schedule wins (rounds of items over the SMs times tiles per item plus one
    // tile's worth of per-item overhead).
    long long best_cost = -1;
    int found = 0;
    for (int nseg = 1; nseg <= g.tw && found < 4; ++nseg) {
        const int txs = (g.tw + nseg - 1) / nseg;
        if (nseg > 1 && txs == (g.tw + nseg - 2) / (nseg - 1)) continue;      // same segment length as before
        const int span = (txs - 1) * g.m + alpha;
        // staged columns: the span, what the vector grid adds in front (up to vec - 1) and what the compute
        // side may read beyond the last tile (whole 4-wide vectors), rounded up to 4 x odd
        int wb = (span + (it->vec - 1) + 3 + 3) / 4 * 4;
        if (((wb / 4) & 1) == 0) wb += 4;
        if (wb > 256) continue;
        if (!tma_ok && alpha * (wb / it->vec) > 32 * kItCopySlots) continue;
        const long long bytes = (long long)alpha * kItChannels * wb * 4;
        long long nbuf = kItSmemBudget / bytes;
        if (nbuf < 3 && !(txs == 1 && nbuf >= 2)) continue;
        if (nbuf > kItMaxBuffers) nbuf = kItMaxBuffers;
        const int real_nseg = (g.tw + txs - 1) / txs;
        const long long n_items = (long long)g.images * g.th * real_nseg * it->cblocks;
        if (n_items >= (1ll << 31)) continue;
        const long long rounds = (n_items + num_sms - 1) / num_sms;
        const long long cost = rounds * (txs + 1);
        ++found;
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            it->txs = txs;
            it->nseg = real_nseg;
            it->wb = wb;
            it->nbuf = (int)nbuf;
            it->buf_words = alpha * kItChannels * wb;
            it->n_items = n_items;
        }
    }
    return best_cost >= 0;
}

// Defined beside the other tensor-map code (contract_umma.cu).
bool encode_input_map(CUtensorMap* map, const float* x, int images, int C, int H, int W, int box_w, bool split_parity);

template <int ALPHA>
cudaError_t launch_input_ws(const float* x, void* V_hi, void* V_lo, const WinoGeom& g, int mode, const TransformMatrices& mats,
                            int* status, int num_sms, cudaStream_t stream)
{
    MatBt2 bt;
    for (int i = 0; i < ALPHA * ALPHA; ++i) bt.v[i] = make_float2(mats.Bt[i], mats.Bt[i]);
    const bool sym = bt_has_symmetric_structure(mats.Bt, ALPHA);
    constexpr bool kPair = ALPHA <= 6;
    InputItems it;
    bool tma_ok = (g.W % 4 == 0) && ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) && (!kPair || g.Cin % 2 == 0);
    CUtensorMap xmap;
    std::memset(&xmap, 0, sizeof(xmap));
    if (tma_ok) {
        if (!plan_input_items(g, ALPHA, true, num_sms, &it) || !encode_input_map(&xmap, x, g.images, g.Cin, g.H, g.W, it.wb, kPair))
            tma_ok = false;
    }
    if (!tma_ok) {
        // small planes: the whole image of a channel block in shared memory
        PlaneItems pi;
        size_t psmem = 0;
        if (plan_plane_items(g, ALPHA, &pi, &psmem)) {
            auto launch_plane = [&](auto kern) -> cudaError_t {
                cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kItSmemBudget);
                if (e != cudaSuccess) return e;
                return launch_overlapped(kern, dim3((unsigned)(g.images * pi.cblocks)), dim3(kItThreads), psmem, stream, x,
                                         static_cast<char*>(V_hi), static_cast<char*>(V_lo), g, pi, mode, bt);
            };
            if (sym) return launch_plane(input_transform_plane_kernel<ALPHA, true, kPair>);
            return launch_plane(input_transform_plane_kernel<ALPHA, false, kPair>);
        }
    }
    if (!tma_ok && !plan_input_items(g, ALPHA, false, num_sms, &it)) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)it.nbuf * it.buf_words * sizeof(float);
    long long grid = it.n_items < num_sms ? it.n_items : num_sms;
    if (grid <= 0) return cudaSuccess;
    auto launch = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kItSmemBudget);
        if (e != cudaSuccess) return e;
        return launch_overlapped(kern, dim3((unsigned)grid), dim3(kItThreads), smem, stream, x, xmap, static_cast<char*>(V_hi),
                                 static_cast<char*>(V_lo), g, it, mode, bt, status);
    };
    if (sym) return launch(input_transform_ws_kernel<ALPHA, true, kPair>);
    return launch(input_transform_ws_kernel<ALPHA, false, kPair>);
}

}  // namespace wino
}  // namespace mnnb
