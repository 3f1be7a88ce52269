"""ORACLE — test infrastructure only (tests, the smoke check and the benchmark's
CPU-baseline leg may import this; the product path never does).

Exact-rational Winograd generator and Winograd convolution (Eq. 6 and Eq. 8).

Construction (Toom-Cook with a point at infinity), in the paper's notation
n = output tile size (called ``m`` here, as in F(m x m, k x k)), k = kernel
size, alpha = m + k - 1:

  * Eq. 8 prints the polynomial  M(x) = x (x-f)(x+f)(x-2f)(x+2f)...  whose roots
    are the finite interpolation points p_0..p_{alpha-2}; the alpha-th point is
    infinity.  (Reading: the first alpha-1 of 0,+f,-f,+2f,-2f,...; the printed
    last factor would give one root too many.)
  * The linear convolution s = g * u of a k-vector and an m-vector has alpha
    coefficients.  Evaluate both at the points, multiply, interpolate:
        s(x) = s_inf M(x) + sum_i s(p_i) prod_{j!=i}(x-p_j) / N_i,
        N_i = prod_{j!=i}(p_i-p_j),   s_inf = g_{k-1} u_{m-1}.
    So  T(g) = C diag(E_k g) E_m  with T(g) the alpha x m Toeplitz matrix of g,
    E_r the alpha x r evaluation matrix (rows [1,p,p^2,..]; infinity row
    [0,..,0,1]) and C the matrix whose columns hold the interpolation
    polynomials' coefficients.
  * The correlation  y_j = sum_i d_{j+i} g_i  is  y = T(g)^T d, hence
        y = A^T [ (G g) (.) (B^T d) ]
    with A = E_m, G = diag(1/N_i) E_k (the 1/N_i may sit on either side) and
    B^T = rows of coefficients of prod_{j!=i}(x-p_j), last row those of M(x).
  * 2-D (Eq. 6):  Y = A^T [ sum_channels (G W G^T) (.) (B^T X B) ] A.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

POINTS_PAPER = 1   # 0, +-1/2, +-1, ...   (f = 1/2, the paper's choice)
POINTS_UNIT = 2    # 0, +-1, +-2, ...     (f = 1)
POINTS_MIXED = 3   # 0, +-1, +-1/2, +-2, +-1/4, +-4


def interpolation_points(alpha: int, points_id: int = POINTS_PAPER) -> list[Fraction]:
    """The alpha-1 finite points (the alpha-th is infinity)."""
    need = alpha - 1
    if need < 0:
        raise ValueError("alpha must be >= 1")
    if points_id in (POINTS_PAPER, POINTS_UNIT):
        f = Fraction(1, 2) if points_id == POINTS_PAPER else Fraction(1)
        seq, j = [Fraction(0)], 1
        while len(seq) < need:
            seq.append(j * f)
            seq.append(-j * f)
            j += 1
    elif points_id == POINTS_MIXED:
        mags = [Fraction(1), Fraction(1, 2), Fraction(2), Fraction(1, 4), Fraction(4),
                Fraction(3, 4), Fraction(4, 3)]
        seq = [Fraction(0)]
        for v in mags:
            seq += [v, -v]
        if need > len(seq):
            raise ValueError("mixed point set has only %d points" % len(seq))
    else:
        raise ValueError("unknown points_id")
    return seq[:need]


def _poly_mul(a, b):
    out = [Fraction(0)] * (len(a) + len(b) - 1)
    for i, ai in enumerate(a):
        for j, bj in enumerate(b):
            out[i + j] += ai * bj
    return out


def generate(m: int, k: int, points_id: int = POINTS_PAPER, points=None):
    """(A, G, Bt) as lists of lists of Fraction: A is alpha x m, G alpha x k,
    Bt alpha x alpha, for F(m, k).  ``points`` overrides the point set."""
    if m < 1 or k < 1:
        raise ValueError("m and k must be >= 1")
    alpha = m + k - 1
    p = [Fraction(v) for v in points] if points is not None else interpolation_points(alpha, points_id)
    if len(p) != alpha - 1 or len(set(p)) != len(p):
        raise ValueError("need alpha-1 distinct finite points")
    zero, one = Fraction(0), Fraction(1)
    A = [[pi ** j for j in range(m)] for pi in p] + [[zero] * (m - 1) + [one]]
    G, Bt = [], []
    for i, pi in enumerate(p):
        Ni, poly = one, [one]
        for j, pj in enumerate(p):
            if j != i:
                Ni *= (pi - pj)
                poly = _poly_mul(poly, [-pj, one])
        G.append([pi ** j / Ni for j in range(k)])
        Bt.append(poly + [zero] * (alpha - len(poly)))
    Mx = [one]
    for pj in p:
        Mx = _poly_mul(Mx, [-pj, one])
    G.append([zero] * (k - 1) + [one])
    Bt.append(Mx)
    return A, G, Bt


def matrices_f64(m, k, points_id=POINTS_PAPER):
    """(At [m x alpha], G [alpha x k], Bt [alpha x alpha]) as float64 arrays."""
    A, G, Bt = generate(m, k, points_id)
    return (np.array([[float(v) for v in r] for r in A], dtype=np.float64).T.copy(),
            np.array([[float(v) for v in r] for r in G], dtype=np.float64),
            np.array([[float(v) for v in r] for r in Bt], dtype=np.float64))


def matrices_f32(m, k, points_id=POINTS_PAPER):
    """The same three matrices, each exact rational rounded once to fp32
    (round-to-nearest-even via float64: every entry here has a short binary or
    small-denominator form, and double rounding cannot occur for a Fraction
    converted by Python's correctly rounded ``float`` then to fp32 unless the
    fp64 value sits on an fp32 tie, which is checked)."""
    A, G, Bt = generate(m, k, points_id)

    def to32(rows):
        out = np.empty((len(rows), len(rows[0])), dtype=np.float32)
        for i, r in enumerate(rows):
            for j, v in enumerate(r):
                out[i, j] = _fraction_to_f32(v)
        return out

    return to32(A).T.copy(), to32(G), to32(Bt)


def _fraction_to_f32(v: Fraction) -> np.float32:
    """Correctly rounded (nearest-even) fp32 of an exact rational."""
    if v == 0:
        return np.float32(0.0)
    d = float(v)                       # correctly rounded to fp64
    f = np.float32(d)
    # guard against double rounding: compare the two fp32 neighbours exactly
    lo = np.nextafter(f, np.float32(-np.inf))
    hi = np.nextafter(f, np.float32(np.inf))
    best, best_err = None, None
    for c in (lo, f, hi):
        err = abs(Fraction(float(c)) - v)
        if best is None or err < best_err:
            best, best_err = c, err
        elif err == best_err:
            # tie: pick the one with an even mantissa
            if (np.float32(c).view(np.uint32) & 1) == 0:
                best = c
    return np.float32(best)


# ---------------------------------------------------------------------------
# Exact evaluation (Fractions) — small inputs only.
# ---------------------------------------------------------------------------
def _matvec(Mx, v):
    return [sum(r[j] * v[j] for j in range(len(v))) for r in Mx]


def winograd_1d_exact(d, g, m, points_id=POINTS_PAPER):
    """y = A^T[(G g) (.) (B^T d)] for one tile: len(d) = alpha, len(g) = k -> m outputs."""
    k = len(g)
    A, G, Bt = generate(m, k, points_id)
    alpha = m + k - 1
    if len(d) != alpha:
        raise ValueError("tile must have alpha entries")
    U = _matvec(G, [Fraction(v) for v in g])
    V = _matvec(Bt, [Fraction(v) for v in d])
    prod = [U[i] * V[i] for i in range(alpha)]
    return [sum(A[i][j] * prod[i] for i in range(alpha)) for j in range(m)]


def _mat_mul(X, Y):
    return [[sum(X[i][t] * Y[t][j] for t in range(len(Y))) for j in range(len(Y[0]))] for i in range(len(X))]


def _transpose(X):
    return [list(r) for r in zip(*X)]


def winograd_2d_tile_exact(X_tiles, W_kernels, m, points_id=POINTS_PAPER):
    """Eq. 6 for one output tile of one output channel.
    X_tiles: list over channels of alpha x alpha tiles; W_kernels: list over
    channels of k x k kernels.  Returns the m x m output tile (Fractions)."""
    k = len(W_kernels[0])
    A, G, Bt = generate(m, k, points_id)
    alpha = m + k - 1
    Gt, B, At = _transpose(G), _transpose(Bt), _transpose(A)
    acc = [[Fraction(0)] * alpha for _ in range(alpha)]
    for X, Wk in zip(X_tiles, W_kernels):
        Xf = [[Fraction(v) for v in r] for r in X]
        Wf = [[Fraction(v) for v in r] for r in Wk]
        U = _mat_mul(_mat_mul(G, Wf), Gt)
        V = _mat_mul(_mat_mul(Bt, Xf), B)
        for i in range(alpha):
            for j in range(alpha):
                acc[i][j] += U[i][j] * V[i][j]
    return _mat_mul(_mat_mul(At, acc), A)


def winograd_conv_exact(x, w, m, pad=0, points_id=POINTS_PAPER):
    """Whole stride-1 convolution of integer arrays through Eq. 6, tiles taken
    from the output side (ceil(OH/m) x ceil(OW/m) tiles per image; input beyond
    the image reads as zero; outputs beyond OH, OW are dropped).
    x [N,C,H,W], w [Co,C,k,k] integer arrays -> nested list [N][Co][OH][OW] of Fraction."""
    x = np.asarray(x)
    w = np.asarray(w)
    N, C, H, W = x.shape
    Co, _, k, _ = w.shape
    alpha = m + k - 1
    OH, OW = H + 2 * pad - k + 1, W + 2 * pad - k + 1
    th, tw = -(-OH // m), -(-OW // m)
    out = [[[[None] * OW for _ in range(OH)] for _ in range(Co)] for _ in range(N)]

    def xat(n, c, i, j):
        return int(x[n, c, i, j]) if 0 <= i < H and 0 <= j < W else 0

    for n in range(N):
        for ty in range(th):
            for tx in range(tw):
                tiles = [[[xat(n, c, ty * m - pad + a, tx * m - pad + b) for b in range(alpha)]
                          for a in range(alpha)] for c in range(C)]
                for co in range(Co):
                    kern = [[[int(w[co, c, a, b]) for b in range(k)] for a in range(k)] for c in range(C)]
                    Y = winograd_2d_tile_exact(tiles, kern, m, points_id)
                    for a in range(m):
                        for b in range(m):
                            oh, ow = ty * m + a, tx * m + b
                            if oh < OH and ow < OW:
                                out[n][co][oh][ow] = Y[a][b]
    return out


# ---------------------------------------------------------------------------
# fp64 stage evaluations (for checking the GPU stages one by one).
# Layouts follow the mathematics, not any device layout: callers reshape.
# ---------------------------------------------------------------------------
def weight_transform_f64(w, m, points_id=POINTS_PAPER):
    """U[xi, co, ci] = (G w[co,ci] G^T)[xi], xi = i*alpha + j, fp64."""
    w = np.asarray(w, dtype=np.float64)
    k = w.shape[2]
    _, G, _ = matrices_f64(m, k, points_id)
    alpha = m + k - 1
    U = np.einsum("ia,ocab,jb->ijoc", G, w, G)
    return U.reshape(alpha * alpha, w.shape[0], w.shape[1])


def extract_tiles_f64(x, m, k, pad):
    """All alpha x alpha input tiles at stride m (zero beyond the image):
    [N, th, tw, C, alpha, alpha] fp64; tiles counted from the output side."""
    x = np.asarray(x, dtype=np.float64)
    N, C, H, W = x.shape
    alpha = m + k - 1
    OH, OW = H + 2 * pad - k + 1, W + 2 * pad - k + 1
    th, tw = -(-OH // m), -(-OW // m)
    Hp, Wp = th * m + k - 1, tw * m + k - 1
    xp = np.zeros((N, C, Hp + pad, Wp + pad), dtype=np.float64)
    xp[:, :, pad:pad + H, pad:pad + W] = x
    xp = xp[:, :, :Hp, :Wp]
    tiles = np.empty((N, th, tw, C, alpha, alpha), dtype=np.float64)
    for ty in range(th):
        for tx in range(tw):
            tiles[:, ty, tx] = xp[:, :, ty * m:ty * m + alpha, tx * m:tx * m + alpha]
    return tiles


def input_transform_f64(x, m, k, pad, points_id=POINTS_PAPER):
    """V[xi, t, ci] = (B^T d B)[xi] with t = (n*th + ty)*tw + tx, fp64."""
    _, _, Bt = matrices_f64(m, k, points_id)
    tiles = extract_tiles_f64(x, m, k, pad)
    N, th, tw, C, alpha, _ = tiles.shape
    V = np.einsum("ia,ntucab,jb->ijntuc", Bt, tiles, Bt)
    return V.reshape(alpha * alpha, N * th * tw, C)


def output_transform_f64(M, m, k, N, OH, OW, bias=None, relu=False, points_id=POINTS_PAPER):
    """y[n,co,ty*m+a,tx*m+b] = act((A^T M A)[a,b] + bias[co]) from
    M[xi, co, t] (t as in input_transform_f64), fp64 [N,Cout,OH,OW]."""
    At, _, _ = matrices_f64(m, k, points_id)
    alpha = m + k - 1
    M = np.asarray(M, dtype=np.float64)
    Co = M.shape[1]
    th, tw = -(-OH // m), -(-OW // m)
    Mr = M.reshape(alpha, alpha, Co, N, th, tw)
    Y = np.einsum("ai,ijontu,bj->notaub", At, Mr, At).reshape(N, Co, th * m, tw * m)[:, :, :OH, :OW]
    if bias is not None:
        Y = Y + np.asarray(bias, dtype=np.float64)[None, :, None, None]
    if relu:
        Y = np.maximum(Y, 0.0)
    return np.ascontiguousarray(Y)


def winograd_conv_f64(x, w, m, pad, bias=None, relu=False, points_id=POINTS_PAPER, operand_round=None):
    """The three stages chained in fp64.  ``operand_round`` (a function applied
    to U and V, e.g. a TF32/BF16 rounding emulation) lets a test see how much
    error reduced-precision operands add; None keeps everything fp64."""
    x = np.asarray(x)
    w = np.asarray(w)
    k = w.shape[2]
    N, _, H, W = x.shape
    OH, OW = H + 2 * pad - k + 1, W + 2 * pad - k + 1
    U = weight_transform_f64(w, m, points_id)
    V = input_transform_f64(x, m, k, pad, points_id)
    if operand_round is not None:
        U, V = operand_round(U), operand_round(V)
    Mm = np.einsum("xoc,xtc->xot", U, V)
    return output_transform_f64(Mm, m, k, N, OH, OW, bias, relu, points_id)


def round_to_mantissa(a, bits):
    """Round-to-nearest-even of fp32(a) to ``bits`` explicit mantissa bits
    (10 = TF32, 7 = BF16), returned as float64.  Finite inputs only."""
    a32 = np.asarray(a, dtype=np.float32)
    u = a32.view(np.uint32).astype(np.uint64)
    drop = 23 - bits
    if drop <= 0:
        return a32.astype(np.float64)
    half = np.uint64(1) << np.uint64(drop - 1)
    lsb = (u >> np.uint64(drop)) & np.uint64(1)
    u = ((u + half - np.uint64(1) + lsb) >> np.uint64(drop)) << np.uint64(drop)
    return u.astype(np.uint32).view(np.float32).astype(np.float64)
