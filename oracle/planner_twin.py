"""ORACLE — test infrastructure only (tests may import this; the product path never does).

Python-integer restatement of the pre-inference planner (Section 3.2, Eq. 1-5).

The paper selects a computation scheme per convolution layer by minimising a cost
(Eq. 1): an arithmetic count (Eq. 2) that picks the Winograd tile size, the rule that
k = 1 is a matrix product and n-hat = 1 means sliding window (Eq. 3), and a backend term
MUL / FLOPS + t_schedule per operator (Eq. 4, 5).  Read for one GPU whose kernels are
bound by memory traffic, tensor throughput or ALU throughput, the cost of a candidate
scheme is the sum over its kernels of

    max(bytes x c_byte, tensor flops x c_tensor, ALU flops x c_alu) // 10^6 + c_launch

in integer picoseconds; the rate constants are attoseconds per unit, measured once on
the GPU and frozen in a record of sixteen integers (the paper's FLOPS and t_schedule
constants, Appendix C).  The candidate with the smallest cost wins; the first one in
the fixed candidate order wins ties.  Candidates whose predicted error exceeds 0.7 x the
tolerance of the accuracy class are not admissible.  The predicted errors are integers
(parts per million) handed in as a table, so that everything here is a function of
integers: nine layer integers, the options, the sixteen constants and that table.

Candidate order (index into cost_ps): 0 direct; 1 GEMM tf32; 2 GEMM bf16; 3-5 Winograd
m = 2, 4, 6 tf32 x1; 6-8 tf32 x3; 9-11 bf16 x1; 12-14 bf16 x3; 15 Winograd F(2x2,3x3) as one
fused kernel (tf32 x1).

Also here: the paper's own multiplication count (Eq. 2) with the two corrections that make
it comparable across tile sizes (it is a per-tile count; its third term lacks the output
channels), reported beside the choice, and an fp64 restatement of the accuracy model.

Python integers are unbounded; the library saturates every picosecond figure at
2^64 - 2 and so does this file, at the same places.
"""
from __future__ import annotations

from dataclasses import dataclass, field

ALGO_WINOGRAD, ALGO_GEMM, ALGO_DIRECT = 1, 2, 3
OPERAND_TF32, OPERAND_BF16, OPERAND_FP32_REF = 1, 2, 3
PREC_TF32, PREC_BF16 = 0, 1
LHS_PATCHES, LHS_X, LHS_IMPLICIT = 1, 2, 3
INADMISSIBLE = 2 ** 64 - 1
SATURATED = 2 ** 64 - 2
MAX_CHUNK_BYTES = 4 << 30          # V + M of one chunk may not exceed this, whatever the cost says
LHS_X_ERROR_PPM = 340              # truncation of x to TF32 by the tensor core itself (measured)
N_CANDIDATES = 16
FUSED_SLOT = 15


def cdiv(a: int, b: int) -> int:
    return -(-a // b)


def sat(v: int) -> int:
    return min(v, SATURATED)


@dataclass(frozen=True)
class Layer:
    N: int
    Cin: int
    Cout: int
    H: int
    W: int
    k: int
    stride: int = 1
    pad: int = 0
    dil: int = 1
    groups: int = 1

    @property
    def OH(self) -> int:
        return (self.H + 2 * self.pad - self.dil * (self.k - 1) - 1) // self.stride + 1

    @property
    def OW(self) -> int:
        return (self.W + 2 * self.pad - self.dil * (self.k - 1) - 1) // self.stride + 1


@dataclass(frozen=True)
class Options:
    precision: int = PREC_TF32
    operand: int = 0
    passes: int = 0
    force_algo: int = 0
    force_m: int = 0
    points_id: int = 0
    gemm_lhs: int = 0
    fused: int = 0            # 0 planner, 1 never, 2 the fused kernel or nothing


@dataclass
class Choice:
    algo: int = 0
    m: int = 0
    operand: int = 0
    passes: int = 0
    points_id: int = 0
    gemm_lhs: int = 0
    chunk_images: int = 0
    n_chunks: int = 0
    fused: int = 0
    chosen: int = -1
    error_ppm: int = 0
    cost_ps: list = field(default_factory=lambda: [INADMISSIBLE] * N_CANDIDATES)


# ---------------------------------------------------------------------------------------
# One kernel: Eq. 5 with three possible bounds and the launch term.
# ---------------------------------------------------------------------------------------
def kernel_ps(c, mem_as: int = 0, tensor_as: int = 0, alu_as: int = 0) -> int:
    return sat(max(mem_as, tensor_as, alu_as) // 1_000_000 + c[5])


def _bytes_of(operand: int) -> int:
    return 2 if operand == OPERAND_BF16 else 4


def _tensor_rate(c, operand: int) -> int:
    return c[3] if operand == OPERAND_BF16 else c[2]


# ---------------------------------------------------------------------------------------
# Sliding window (Section 3.2 item 3): one kernel, input + output + weights once.
# ---------------------------------------------------------------------------------------
def direct_cost(L: Layer, c) -> int:
    cpg = L.Cin // L.groups
    traffic = 4 * (L.N * L.Cin * L.H * L.W + L.N * L.Cout * L.OH * L.OW + L.Cout * cpg * L.k * L.k)
    flops = 2 * L.N * L.Cout * cpg * L.OH * L.OW * L.k * L.k
    # layers with at most four input channels have a kernel of their own with its own rate,
    # when its transposed weights fit 160 KiB of shared memory
    few_channels = (L.groups == 1 and L.Cin <= 4 and c[9] > 0 and L.N <= 65535
                    and L.Cin * L.k * L.k * (cdiv(L.Cout, 32) * 32) * 4 <= 160 * 1024)
    # c[9] is the rate of the 3 -> Cout, 3x3, stride 2, padding 1 layer on even H and W a multiple of 4 (weights
    # within 48 KiB), which has its own kernel; the other few-channel shapes run at half that rate
    fast = (L.Cin == 3 and L.k == 3 and L.stride == 2 and L.pad == 1 and L.dil == 1 and L.H % 2 == 0 and L.W % 4 == 0
            and 27 * (cdiv(L.Cout, 32) * 32) * 4 <= 48 * 1024)
    rate = (c[9] if fast else 2 * c[9]) if few_channels else c[8]
    return kernel_ps(c, mem_as=traffic * c[0], alu_as=flops * rate)


# ---------------------------------------------------------------------------------------
# Tiling of the tensor-core contraction: output channels per work item.
# ---------------------------------------------------------------------------------------
def contraction_tiling(tile_blocks: int, positions: int, Cout: int, sms: int):
    """(bn, channel blocks): bn a multiple of 16, at most 256, blocks balanced; among 1x, 2x, 4x the minimum
    number of channel blocks the one with the shortest schedule (rounds over the SMs x operand rows per item)."""
    co16 = cdiv(Cout, 16) * 16
    fewest = cdiv(co16, 256)
    best = None
    for mult in (1, 2, 4):
        bn = cdiv(co16 // 16, fewest * mult) * 16
        if bn < 32 and mult > 1:
            break
        blocks = cdiv(co16, bn)
        length = cdiv(tile_blocks * blocks * positions, sms) * (128 + bn)
        if best is None or length < best[0]:
            best = (length, bn, blocks)
    return best[1], best[2]


# ---------------------------------------------------------------------------------------
# GEMM scheme (k = 1 "is just a matrix multiplication"; k > 1 over gathered patches).
# ---------------------------------------------------------------------------------------
def gemm_may_read_x(L: Layer, operand: int, passes: int) -> bool:
    return (L.k == 1 and L.stride == 1 and L.pad == 0 and L.groups == 1 and operand == OPERAND_TF32
            and passes == 1 and L.H * L.W >= 32 and (L.H * L.W) % 4 == 0)


def gemm_cost(L: Layer, operand: int, lhs, c) -> int:
    """lhs: LHS_PATCHES (gather kernel + GEMM), LHS_X / True (the GEMM reads x itself), LHS_IMPLICIT (the patches are
    gathered by producer warps inside the GEMM kernel)."""
    lhs_x = lhs is True or lhs == LHS_X
    implicit = lhs is not True and lhs == LHS_IMPLICIT
    b = _bytes_of(operand)
    Kp = cdiv(L.Cin * L.k * L.k, 8) * 8
    T = L.N * L.OH * L.OW
    x_bytes = 4 * L.N * L.Cin * L.H * L.W
    y_bytes = 4 * L.N * L.Cout * L.OH * L.OW
    v_bytes = T * Kp * b
    u_bytes = L.Cout * Kp * b
    sms = c[7] if c[7] > 0 else 148
    # the contraction as it is scheduled: rounds of work items, each a serial loop over 128-byte blocks of K
    # paced by the tensor core or by the delivery of the operand tiles (16 ps per byte), the accumulator drained
    # (45 ps per byte, half a microsecond of hand-over) while the next item's loop runs; one drain is exposed
    tile_blocks = L.N * cdiv(cdiv(L.H * L.W, 32), 4) if lhs_x else cdiv(T, 128)
    bn, co_blocks = contraction_tiling(tile_blocks, 1, L.Cout, sms)
    rounds = cdiv(tile_blocks * co_blocks, sms)
    k_elems = 128 // b
    k_blocks = cdiv(Kp, k_elems)
    deliver_ps = (128 * 128 + bn * 128) * 16
    mma_ps = sat(2 * 128 * bn * k_elems * _tensor_rate(c, operand) * sms // 1_000_000)
    drain_ps = 128 * bn * 4 * 45
    if implicit:
        # only the weight tile is delivered; the gather of 128 x 32 patch elements (c[13] attoseconds each) paces a block too
        # (c[13] is measured on the tap-major gather, Cin a multiple of 32; other channel counts gather element-wise, about 2x)
        block_ps = max(bn * 128 * 16, mma_ps, sat(128 * 32 * c[13] * (1 if L.Cin % 32 == 0 else 2) // 1_000_000))
        item_i = max(k_blocks * block_ps, drain_ps + 500_000)
        return kernel_ps(c, mem_as=(x_bytes + u_bytes + y_bytes) * c[0], tensor_as=(rounds * item_i + drain_ps) * 1_000_000)
    item_ps = max(k_blocks * max(deliver_ps, mma_ps), drain_ps + 500_000)
    serial_as = (rounds * item_ps + drain_ps) * 1_000_000
    if lhs_x:
        return kernel_ps(c, mem_as=(x_bytes + u_bytes + y_bytes) * c[0], tensor_as=serial_as)
    # the patch gather at its measured rate relative to a plain copy: 1.5x (1x1 stride-1: a transposition),
    # 3x (k > 1, staged through shared memory), 5x (strided 1x1, element-wise)
    transposition = L.k == 1 and L.stride == 1 and L.pad == 0 and (L.H * L.W) % 4 == 0
    twice_factor = 3 if transposition else (6 if L.k > 1 else 10)
    gather = kernel_ps(c, mem_as=(x_bytes + v_bytes) * c[0] * twice_factor // 2)
    contract = kernel_ps(c, mem_as=(v_bytes + u_bytes + y_bytes) * c[0], tensor_as=serial_as)
    return sat(gather + contract)


# ---------------------------------------------------------------------------------------
# Winograd F(m x m, k x k) as three kernels (Eq. 6), chunked over the batch.
# ---------------------------------------------------------------------------------------
def winograd_supported(m: int, k: int) -> bool:
    return m in (2, 4, 6) and k in (2, 3, 5, 7) and m + k - 1 <= 12


def winograd_cost(L: Layer, m: int, operand: int, passes: int, c):
    """(chunk_images, n_chunks, cost_ps)."""
    alpha = m + L.k - 1
    a2 = alpha * alpha
    tiles_img = cdiv(L.OH, m) * cdiv(L.OW, m)
    Cp = cdiv(L.Cin, 8) * 8
    b_el = _bytes_of(operand) * (2 if passes == 3 else 1)
    per_image = a2 * tiles_img * Cp * b_el + a2 * L.Cout * tiles_img * 4
    fits_l2 = c[6] // per_image
    cap = max(1, MAX_CHUNK_BYTES // per_image)
    chunk = L.N if L.N < cap else cdiv(L.N, cdiv(L.N, cap))
    n_chunks = cdiv(L.N, chunk)
    # one chunk: input transform, contraction, output transform
    n = chunk
    v = n * a2 * tiles_img * Cp * b_el
    mm = n * a2 * L.Cout * tiles_img * 4
    u = a2 * L.Cout * Cp * b_el
    x = 4 * n * L.Cin * L.H * L.W
    y = 4 * n * L.Cout * L.OH * L.OW
    c_vm = c[1] if fits_l2 >= chunk else c[0]
    # ALU work of the transforms: 2 alpha^3 multiply-adds per (tile, channel) on the input side (the first term
    # of Eq. 2), m alpha (alpha + m) on the output side (its third term); from alpha = 8 a lane holds one channel
    # instead of a pair and sweeps over the tile's columns: x2 at alpha = 8, x2.25 at alpha = 10, x4 at alpha = 12
    # (in quarters: 8, 9, 16 against 4)
    quarters = 16 if alpha >= 12 else (9 if alpha >= 10 else (8 if alpha >= 8 else 4))
    t_in = kernel_ps(c, mem_as=x * c[0] + v * c_vm, alu_as=quarters * alpha * a2 * n * tiles_img * L.Cin * c[4])
    # the contraction's work items (128 tiles x bn channels x one position) go over the SMs in rounds, and the
    # tensor time is that of full rounds
    sms = c[7] if c[7] > 0 else 148
    tile_blocks = cdiv(n * tiles_img, 128)
    _, co_blocks = contraction_tiling(tile_blocks, a2, L.Cout, sms)
    items = tile_blocks * co_blocks * a2
    tensor = 2 * a2 * L.Cout * Cp * n * tiles_img * passes * _tensor_rate(c, operand) // items * (cdiv(items, sms) * sms)
    t_con = kernel_ps(c, mem_as=(v + mm) * c_vm + u * c[0], tensor_as=tensor)
    t_out = kernel_ps(c, mem_as=mm * c_vm + y * c[0], alu_as=2 * m * alpha * (alpha + m) * n * tiles_img * L.Cout * c[4])
    return chunk, n_chunks, sat(n_chunks * sat(t_in + t_con + t_out))


# ---------------------------------------------------------------------------------------
# Winograd F(2x2, 3x3) as ONE kernel: transforms in the producer and epilogue warps, the sixteen
# accumulators of a block of 128 output channels x 32 tiles in tensor memory.  HBM sees x, y and U only.
# ---------------------------------------------------------------------------------------
def fused_supported(L: Layer) -> bool:
    return L.k == 3 and L.stride == 1 and L.dil == 1 and L.groups == 1 and L.pad <= 2


def fused_cost(L: Layer, c) -> int:
    tiles = L.N * cdiv(L.OH, 2) * cdiv(L.OW, 2)
    sms = c[7] if c[7] > 0 else 148
    x = 4 * L.N * L.Cin * L.H * L.W
    y = 4 * L.N * L.Cout * L.OH * L.OW
    u = 16 * L.Cout * L.Cin * 4
    co_blocks = cdiv(L.Cout, 128)
    items = cdiv(tiles, 32) * co_blocks
    rounds = cdiv(items, sms)
    k_blocks = cdiv(L.Cin, 32)
    # an item is a serial loop over blocks of 32 input channels; a block costs the delivery of sixteen
    # 128 x 32 weight tiles from L2 to the SM (c[10] attoseconds per byte and SM) or sixty-four small MMAs
    # whose pace the shared-memory reads of the 128-row operand set (c[11] picoseconds per block), whichever
    # is larger; then the epilogue (c[12] picoseconds per item) before the next item's MMAs may start
    block_ps = max(16 * 128 * 32 * 4 * c[10] // 1_000_000, c[11])
    item_ps = k_blocks * block_ps + c[12]
    serial_as = rounds * item_ps * 1_000_000
    # x comes from HBM once; the other channel blocks find it in L2
    return kernel_ps(c, mem_as=(x + y + u) * c[0] + (co_blocks - 1) * x * c[1], tensor_as=serial_as)


# ---------------------------------------------------------------------------------------
# The selection (Eq. 1, Eq. 3).
# ---------------------------------------------------------------------------------------
def _candidates():
    out = [(ALGO_DIRECT, 0, 0, 0), (ALGO_GEMM, 0, OPERAND_TF32, 1), (ALGO_GEMM, 0, OPERAND_BF16, 1)]
    for operand, passes in ((OPERAND_TF32, 1), (OPERAND_TF32, 3), (OPERAND_BF16, 1), (OPERAND_BF16, 3)):
        for m in (2, 4, 6):
            out.append((ALGO_WINOGRAD, m, operand, passes))
    out.append((ALGO_WINOGRAD, 2, OPERAND_TF32, 1))       # slot 15: the fused kernel
    return out


def best_points(ppm, m, k, operand, passes):
    """(points_id, ppm) with the lowest predicted error; the first wins ties.  ``ppm`` maps
    (m, k, points_id, operand, passes) to parts per million, missing or negative = not available."""
    best = (0, -1)
    for pid in (1, 2, 3):
        p = ppm.get((m, k, pid, operand, passes), -1)
        if p < 0:
            continue
        if best[0] == 0 or p < best[1]:
            best = (pid, p)
    return best


def plan(L: Layer, o: Options, c, ppm) -> Choice:
    """The planner's decision for the list-driven case (no off-list forced combination)."""
    ch = Choice()
    gate = (10000 if o.precision == PREC_BF16 else 1000) * 7 // 10
    fully_forced = o.force_m != 0 and o.operand != 0 and o.passes != 0
    wino_shape = L.stride == 1 and L.dil == 1 and L.groups == 1 and 2 <= L.k <= 7
    side = {}
    for i, (algo, m, operand, passes) in enumerate(_candidates()):
        if o.fused == 2 and i != FUSED_SLOT:
            continue
        if o.force_algo != 0 and o.force_algo != algo:
            continue
        if algo == ALGO_DIRECT:
            if o.operand in (0, OPERAND_FP32_REF) or o.force_algo == ALGO_DIRECT:
                ch.cost_ps[i] = direct_cost(L, c)
            continue
        if o.operand != 0 and o.operand != operand:
            continue
        if o.passes != 0 and o.passes != passes:
            continue
        if algo == ALGO_GEMM:
            if L.groups != 1 or o.force_m != 0:
                continue
            p = ppm.get((1, L.k, 0, operand, passes), -1)
            if p < 0:
                continue
            if p > gate and not (o.operand != 0 and o.force_algo == ALGO_GEMM):
                continue
            x_ok = gemm_may_read_x(L, operand, passes)
            implicit_ok = operand == OPERAND_TF32 and passes == 1
            if o.gemm_lhs == LHS_X and not x_ok:
                continue
            if o.gemm_lhs == LHS_IMPLICIT and not implicit_ok:
                continue
            costs = {LHS_PATCHES: gemm_cost(L, operand, LHS_PATCHES, c)}
            if x_ok:
                costs[LHS_X] = gemm_cost(L, operand, LHS_X, c)
            if implicit_ok:
                costs[LHS_IMPLICIT] = gemm_cost(L, operand, LHS_IMPLICIT, c)
            # left operand: as asked for, else the cheapest that applies (patch matrix, x itself, implicit gather;
            # earlier in this order on ties; the implicit gather only once its rate constant is known)
            lhs = o.gemm_lhs
            if lhs == 0:
                lhs = LHS_PATCHES
                if x_ok and costs[LHS_X] < costs[lhs]:
                    lhs = LHS_X
                # (plain pointwise layers keep the tuned paths: measured, the implicit gather never beat them there)
                if implicit_ok and not (L.k == 1 and L.stride == 1) and c[13] > 0 and costs[LHS_IMPLICIT] < costs[lhs]:
                    lhs = LHS_IMPLICIT
            if lhs == LHS_X:
                p = max(p, LHS_X_ERROR_PPM)
            side[i] = dict(lhs=lhs, ppm=p)
            ch.cost_ps[i] = costs[lhs]
            continue
        # Winograd
        fused = i == FUSED_SLOT
        if fused and (o.fused == 1 or not fused_supported(L) or c[10] <= 0 or c[11] <= 0):
            continue
        if not wino_shape or not winograd_supported(m, L.k):
            continue
        if o.force_m != 0 and o.force_m != m:
            continue
        if o.points_id == 0:
            pid, p = best_points(ppm, m, L.k, operand, passes)
        else:
            pid, p = o.points_id, ppm.get((m, L.k, o.points_id, operand, passes), -1)
        if pid == 0 or p < 0:
            continue
        if p > gate and not fully_forced:
            continue
        if fused:
            side[i] = dict(pid=pid, ppm=p, chunk=L.N, n_chunks=1)
            ch.cost_ps[i] = fused_cost(L, c)
        else:
            chunk, n_chunks, cost = winograd_cost(L, m, operand, passes, c)
            side[i] = dict(pid=pid, ppm=p, chunk=chunk, n_chunks=n_chunks)
            ch.cost_ps[i] = cost
    best = -1
    for i in range(N_CANDIDATES):
        if ch.cost_ps[i] != INADMISSIBLE and (best < 0 or ch.cost_ps[i] < ch.cost_ps[best]):
            best = i
    if best < 0:
        return ch
    algo, m, operand, passes = _candidates()[best]
    ch.chosen, ch.algo, ch.operand, ch.passes = best, algo, operand, passes
    ch.error_ppm = side.get(best, {}).get("ppm", 0)
    if algo == ALGO_WINOGRAD:
        ch.m, ch.points_id = m, side[best]["pid"]
        ch.chunk_images, ch.n_chunks = side[best]["chunk"], side[best]["n_chunks"]
        ch.fused = 1 if best == FUSED_SLOT else 0
    else:
        ch.m, ch.points_id, ch.chunk_images, ch.n_chunks = 1, 0, L.N, 1
        ch.gemm_lhs = side[best]["lhs"] if algo == ALGO_GEMM else 0
    return ch


# ---------------------------------------------------------------------------------------
# The paper's own count (Eq. 2), made comparable across n: it is a per-tile count, so it is multiplied by
# the number of tiles, and its third term (the output transform) gets the o_c factor it lacks as printed.
# ---------------------------------------------------------------------------------------
def paper_multiplications(L: Layer, n: int) -> int:
    a = n + L.k - 1
    tiles = L.N * cdiv(L.OH, n) * cdiv(L.OW, n)
    return tiles * (2 * L.Cin * a ** 3 + L.Cin * L.Cout * a ** 2 + L.Cout * n * a * (2 * n + L.k - 1))


def paper_choice(L: Layer, sizes=(1, 2, 4, 6)):
    """(n-hat, [count per n]): Eq. 2's argmin over the tile sizes; n-hat = 1 means sliding window (Eq. 3)."""
    counts = [paper_multiplications(L, n) for n in sizes]
    return sizes[counts.index(min(counts))], counts


# ---------------------------------------------------------------------------------------
# Accuracy model: F(m, k) on a fixed pseudo-random problem in fp64 with U and V rounded to the operand
# format (optionally split into hi + lo), relative L2 error against the plain correlation, in ppm.
# Same data recipe as the library's gate (a 64-bit LCG, sums of twelve uniforms), restated with NumPy.
# ---------------------------------------------------------------------------------------
def _lcg_normalish(seed: int, count: int):
    import numpy as np
    s = seed
    out = np.empty(count, dtype=np.float64)
    mask = (1 << 64) - 1
    for i in range(count):
        acc = 0.0
        for _ in range(12):
            s = (s * 6364136223846793005 + 1442695040888963407) & mask
            acc += (s >> 11) * (1.0 / 9007199254740992.0)
        out[i] = acc - 6.0
    return out


def _round_bits(a, bits):
    """fp32(a) rounded to `bits` explicit mantissa bits, ties to even, as fp64."""
    import numpy as np
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    drop = 23 - bits
    if drop > 0:
        lsb = (u >> np.uint64(drop)) & np.uint64(1)
        u = u + np.uint64((1 << (drop - 1)) - 1) + lsb
        u = u & ~np.uint64((1 << drop) - 1)
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def accuracy_ppm(m: int, k: int, points_id: int, operand: int, passes: int, generate=None) -> int:
    """``generate(m, k, points_id)`` returns (A, G, Bt) as exact rationals (the oracle's generator)."""
    import math

    import numpy as np
    bits = {OPERAND_TF32: 10, OPERAND_BF16: 7, OPERAND_FP32_REF: 23}[operand]
    C, CO, TILES = 64, 4, 16
    alpha = m + k - 1
    a2 = alpha * alpha
    seed = 0x9E3779B97F4A7C15 ^ (m * 1000 + k * 10)
    draws = _lcg_normalish(seed, CO * C * k * k + TILES * C * a2)
    w = (draws[:CO * C * k * k] * (1.0 / math.sqrt(C * k * k))).astype(np.float32).astype(np.float64).reshape(CO, C, k, k)
    x = draws[CO * C * k * k:].astype(np.float32).astype(np.float64).reshape(TILES, C, alpha, alpha)

    def split(v):
        hi = _round_bits(v, bits)
        lo = _round_bits(v.astype(np.float32).astype(np.float64) - hi, bits) if passes == 3 else np.zeros_like(hi)
        return hi, lo

    if m == 1 and points_id == 0:
        wk = w.reshape(CO, C * k * k)              # alpha = k here: a tile is one k x k patch
        xk = x.reshape(TILES, C * k * k)
        wh, wl = split(wk)
        xh, xl = split(xk)
        ref = xk @ wk.T
        got = xh @ wh.T + xh @ wl.T + xl @ wh.T
    else:
        A, G, Bt = generate(m, k, points_id)
        A = np.array([[float(v) for v in r] for r in A])
        G = np.array([[float(v) for v in r] for r in G])
        Bt = np.array([[float(v) for v in r] for r in Bt])
        U = np.einsum("ia,ocab,jb->ocij", G, w, G)
        V = np.einsum("ia,tcab,jb->tcij", Bt, x, Bt)
        Uh, Ul = split(U)
        Vh, Vl = split(V)
        M = (np.einsum("ocij,tcij->toij", Uh, Vh) + np.einsum("ocij,tcij->toij", Ul, Vh)
             + np.einsum("ocij,tcij->toij", Uh, Vl))
        M = M.astype(np.float32).astype(np.float64)
        got = np.einsum("ia,toij,jb->toab", A, M, A)
        ref = np.zeros((TILES, CO, m, m))
        for i in range(k):
            for j in range(k):
                ref += np.einsum("oc,tcab->toab", w[:, :, i, j], x[:, :, i:i + m, j:j + m])
    rel = math.sqrt(float(((got - ref) ** 2).sum()) / float((ref ** 2).sum()))
    return int(math.ceil(rel * 1e6))


# ---------------------------------------------------------------------------------------
# Strassen's stopping rule (Eq. 9) for [n x k] x [k x m]: recurse while the multiplications saved outnumber
# the additions added, both counted alike.
# ---------------------------------------------------------------------------------------
def strassen_rule(m: int, n: int, k: int) -> bool:
    if min(m, n, k) < 2:
        return False
    mh, nh, kh = m // 2, n // 2, k // 2
    return m * n * k - 7 * mh * nh * kh > 4 * mh * kh + 4 * nh * kh + 7 * mh * nh
