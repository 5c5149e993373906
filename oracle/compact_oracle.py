"""CPU oracle for the CompAct compressed linear layer (test infrastructure).

A plain, slow, fp64 restatement of what the layer computes, written from the
paper's Algorithms 1-3 (forward, backward, Adam update step with CompAct) and
Section 3.3 (random projection matrix).  It exists only to check the CUDA
path: tests, the smoke check and the benchmark's CPU-baseline leg may import
it; the product path never does.  It shares no code with the CUDA sources.

Every floating-point step is fp64.  Matrix products call numpy's fp64 matmul
(a library primitive standing for the sum in the definition); there is no
blocking, fusion or reordering beyond what the algorithms state.

Two modes:
  * "exact": no storage rounding anywhere (comparison target for fp32 runs);
  * "bf16" : tensors that the method stores in bfloat16 are rounded to
             nearest-even at exactly these points: P, Y, Z, dX, N, W.

Readings of the paper taken here (the paper is silent or inconsistent):
  * P_ij ~ N(0, 1/r) means variance 1/r (only this gives E[P P^T] = I).
  * P is n x r (it multiplies x of shape bl x n on the right).
  * Adam follows Algorithm 3 (bias correction, sqrt(V)+eps); the bias-corrected
    moments are temporaries and the stored moments are the uncorrected ones;
    the step count used for bias correction is 1-based.
  * The generator behind "set_random_seed(s); P <- N(0,1/r)" is Philox4x32-10
    keyed by the 64-bit seed with counter (j>>3, i, layer, epoch), followed by
    Box-Muller with 16 bits per uniform, so that one call yields the eight
    entries P[i, 8q .. 8q+7]: the entries are stored with eight significant bits
    in bf16 layers, and a generator that spends a whole 32-bit word per uniform
    pays twice the integer work per entry for resolution nobody reads (radii
    reach 4.85 standard deviations instead of 5.77).  The seed bump
    "s <- s+1" is the epoch word.
  * The sparse Johnson-Lindenstrauss projection of the ablation study is the
    construction the paper cites there (Dasgupta, Kumar, Sarlos: each input
    coordinate is hashed s times into the r output coordinates with random
    signs, scaled by 1/sqrt(s); terms that collide add).  Here term t of row i
    of P is word t&3 of the Philox call with counter
    (0x80000000 | t>>2, i, layer, epoch): sign = bit 31, column =
    ((word & 0x7fffffff) * r) >> 31.  Its entries are multiples of 1/sqrt(s)
    and are not rounded in bf16 mode (the device keeps the integer counts in
    its tiles and scales the accumulated sums).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

# ----------------------------------------------------------------------------
# Philox4x32-10 (Salmon et al., SC'11).  Integer-only; results are exact.
# ----------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(ctr, key):
    """Ten-round Philox on arrays of counters.

    ctr: integer array (..., 4), key: integer array broadcastable to (..., 2).
    Returns uint32 array (..., 4).
    """
    ctr = np.asarray(ctr, dtype=np.uint64)
    key = np.asarray(key, dtype=np.uint64)
    c0, c1, c2, c3 = (ctr[..., i] & _MASK32 for i in range(4))
    k0 = key[..., 0] & _MASK32
    k1 = key[..., 1] & _MASK32
    for rnd in range(10):
        p0 = _PHILOX_M0 * c0            # 32x32 -> 64 bit product
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + np.uint64(_PHILOX_W0)) & _MASK32
        k1 = (k1 + np.uint64(_PHILOX_W1)) & _MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def projection_words(seed: int, layer_id: int, epoch: int, n: int, r: int) -> np.ndarray:
    """The raw Philox stream behind P: uint32 array (n, 4*ceil(r/8)).

    Word (i, 4*q + w) is output word w of the call with counter
    (q, i, layer_id, epoch) and key (seed low half, seed high half); it makes
    the entries P[i, 8q + 2w] and P[i, 8q + 2w + 1].
    """
    groups = (r + 7) // 8
    i = np.arange(n, dtype=np.uint64)[:, None]
    q = np.arange(groups, dtype=np.uint64)[None, :]
    ctr = np.empty((n, groups, 4), dtype=np.uint64)
    ctr[..., 0] = q
    ctr[..., 1] = i
    ctr[..., 2] = np.uint64(layer_id & 0xFFFFFFFF)
    ctr[..., 3] = np.uint64(epoch & 0xFFFFFFFF)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint64)
    return philox4x32_10(ctr, key).reshape(n, groups * 4)


def box_muller_from_words(words: np.ndarray) -> np.ndarray:
    """Standard normals from a (..., k) uint32 stream, two per word: (..., 2k).

    The low half of a word gives u1 = ((x & 0xffff) + 0.5) / 2^16 in (0,1), its
    high half u2 = (x >> 16) / 2^16 in [0,1); the word makes the pair
    (rad cos(2 pi u2), rad sin(2 pi u2)) with rad = sqrt(-2 ln u1).
    """
    w = np.asarray(words, dtype=np.uint32)
    u1 = ((w & np.uint32(0xFFFF)).astype(np.float64) + 0.5) * 2.0 ** -16
    u2 = (w >> np.uint32(16)).astype(np.float64) * 2.0 ** -16
    rad = np.sqrt(-2.0 * np.log(u1))
    ang = 2.0 * np.pi * u2
    out = np.stack([rad * np.cos(ang), rad * np.sin(ang)], axis=-1)
    return out.reshape(w.shape[:-1] + (2 * w.shape[-1],))


def sparse_jl_terms(seed: int, layer_id: int, epoch: int, n: int, r: int, s: int):
    """The s hashed terms of every row of a sparse JL projection (Ablation Study, "Sparse
    Johnson-Lindenstrauss (JL) Projection Matrices"): integer arrays (cols, signs) of shape (n, s)
    with cols in [0, r) and signs in {+1, -1}.  Term t of row i comes from word t & 3 of the
    Philox call with counter (0x80000000 | t >> 2, i, layer_id, epoch)."""
    calls = (s + 3) // 4
    i = np.arange(n, dtype=np.uint64)[:, None]
    q = np.arange(calls, dtype=np.uint64)[None, :]
    ctr = np.empty((n, calls, 4), dtype=np.uint64)
    ctr[..., 0] = np.uint64(0x80000000) | q
    ctr[..., 1] = i
    ctr[..., 2] = np.uint64(layer_id & 0xFFFFFFFF)
    ctr[..., 3] = np.uint64(epoch & 0xFFFFFFFF)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint64)
    words = philox4x32_10(ctr, key).reshape(n, calls * 4)[:, :s].astype(np.uint64)
    cols = ((words & np.uint64(0x7FFFFFFF)) * np.uint64(r)) >> np.uint64(31)
    signs = 1 - 2 * (words >> np.uint64(31)).astype(np.int64)
    return cols.astype(np.int64), signs


def projection_sparse_jl(seed: int, layer_id: int, epoch: int, n: int, r: int, s: int) -> np.ndarray:
    """P (n x r) with P[i, j] = (1/sqrt(s)) * sum over the terms of row i that hash to column j of their signs."""
    cols, signs = sparse_jl_terms(seed, layer_id, epoch, n, r, s)
    K = np.zeros((n, r), dtype=np.float64)
    for i in range(n):
        for t in range(s):
            K[i, cols[i, t]] += signs[i, t]
    return K / math.sqrt(s)


def projection(seed: int, layer_id: int, epoch: int, n: int, r: int, mode: str = "exact", sparse_s: int = 0) -> np.ndarray:
    """P (n x r): Algorithm 1 lines 1-2, Algorithm 3 lines 6-7.  sparse_s == 0: entries N(0, 1/r);
    sparse_s > 0: the sparse JL projection with sparse_s terms per row."""
    if sparse_s > 0:
        return projection_sparse_jl(seed, layer_id, epoch, n, r, sparse_s)
    g = box_muller_from_words(projection_words(seed, layer_id, epoch, n, r))[:, :r]
    P = g / math.sqrt(r)
    return round_bf16(P) if mode == "bf16" else P


# ----------------------------------------------------------------------------
# bfloat16 storage rounding (round-to-nearest-even straight from fp64)
# ----------------------------------------------------------------------------
_BF16_MAX = float((2.0 - 2.0 ** -7) * 2.0 ** 127)


def round_bf16(x) -> np.ndarray:
    """Nearest bfloat16 value (ties to even) of each fp64 entry, returned as fp64."""
    x = np.asarray(x, dtype=np.float64)
    out = x.copy()
    fin = np.isfinite(x) & (x != 0.0)
    if not fin.any():
        return out
    xf = x[fin]
    _, e = np.frexp(xf)                       # xf = mant * 2^e, mant in [0.5, 1)
    q = np.maximum(e - 8, -133)               # 8 significant bits; subnormal quantum 2^-133
    y = np.ldexp(np.rint(np.ldexp(xf, -q)), q)
    y = np.where(np.abs(y) > _BF16_MAX, np.copysign(np.inf, y), y)
    out[fin] = y
    return out


def _store(x: np.ndarray, mode: str) -> np.ndarray:
    return round_bf16(x) if mode == "bf16" else x


# ----------------------------------------------------------------------------
# Algorithms 1-3
# ----------------------------------------------------------------------------
def linear_fwd(X: np.ndarray, W: np.ndarray, P: np.ndarray, mode: str = "exact"):
    """Algorithm 1: o = x W and z = x P.  Returns (Y, Z); row t of Z is token t."""
    X = np.asarray(X, dtype=np.float64)
    Y = X @ np.asarray(W, dtype=np.float64)
    Z = X @ np.asarray(P, dtype=np.float64)
    return _store(Y, mode), _store(Z, mode)


def linear_bwd(dY: np.ndarray, Z: np.ndarray, W: np.ndarray, mode: str = "exact"):
    """Algorithm 2: G_hat = z^T dL/do (r x m, never rounded) and dL/dx = dL/do W^T."""
    dY = np.asarray(dY, dtype=np.float64)
    Gc = np.asarray(Z, dtype=np.float64).T @ dY
    dX = dY @ np.asarray(W, dtype=np.float64).T
    return _store(dX, mode), Gc


def linear_bwd_recompute(X: np.ndarray, dY: np.ndarray, W: np.ndarray, P: np.ndarray, mode: str = "exact"):
    """Algorithm 2 when no z was kept (the combination with activation checkpointing proposed in the
    Limitations section): z = x P is formed again from the recomputed x, as line 4 of Algorithm 1 does,
    and then the two products of Algorithm 2 follow."""
    Z = _store(np.asarray(X, dtype=np.float64) @ np.asarray(P, dtype=np.float64), mode)
    return linear_bwd(dY, Z, W, mode)


def group_fwd(X: np.ndarray, Ws, Ps, mode: str = "exact"):
    """Algorithm 1 for layers that share their input x (q, k, v; gate, up): each layer g has its own W_g and its
    own P_g, and keeps its own z_g = x P_g (appendix on saved tensors, Table 6)."""
    outs = [linear_fwd(X, W, P, mode) for W, P in zip(Ws, Ps)]
    return [o[0] for o in outs], [o[1] for o in outs]


def group_bwd(dYs, Zs, Ws, mode: str = "exact"):
    """Algorithm 2 for such a group: G_hat_g = z_g^T dL/do_g per layer, and the gradient with respect to the shared
    input is the sum of the layers' contributions, dL/dx = sum_g dL/do_g W_g^T (stored once)."""
    Gcs = [np.asarray(Z, dtype=np.float64).T @ np.asarray(dY, dtype=np.float64) for dY, Z in zip(dYs, Zs)]
    dX = sum(np.asarray(dY, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T for dY, W in zip(dYs, Ws))
    return _store(dX, mode), Gcs


def adam_update(W, Gc, M, V, t: int, P, lr: float, beta1: float, beta2: float, eps: float,
                alpha: float = 1.0, mode: str = "exact"):
    """Algorithm 3 lines 1-9 for the update whose 1-based count is t.

    Returns (W_next, M_next, V_next); the returned moments are the uncorrected
    running averages.
    """
    Gc = np.asarray(Gc, dtype=np.float64)
    M = beta1 * np.asarray(M, dtype=np.float64) + (1.0 - beta1) * Gc
    V = beta2 * np.asarray(V, dtype=np.float64) + (1.0 - beta2) * Gc * Gc
    M_hat = M / (1.0 - beta1 ** t)
    V_hat = V / (1.0 - beta2 ** t)
    N = _store(M_hat / (np.sqrt(V_hat) + eps), mode)
    G_tilde = alpha * (np.asarray(P, dtype=np.float64) @ N)
    W_next = np.asarray(W, dtype=np.float64) - lr * G_tilde
    return _store(W_next, mode), M, V


@dataclass
class LayerState:
    """Seed, step and refresh bookkeeping of one layer (Algorithm 3 lines 10-13)."""
    seed: int
    layer_id: int
    refresh_T: int          # 0: never refresh
    epoch: int = 0
    step: int = 0

    def advance(self) -> None:
        """t <- t+1; every T-th update bumps the seed (here: the epoch word)."""
        self.step += 1
        if self.refresh_T > 0 and self.step % self.refresh_T == 0:
            self.epoch += 1


class CompActLayerOracle:
    """One layer's W, M, V and schedule, stepping through Algorithms 1-3."""

    def __init__(self, W0, n: int, m: int, r: int, seed: int, layer_id: int, refresh_T: int,
                 lr: float, beta1: float, beta2: float, eps: float, alpha: float = 1.0,
                 mode: str = "exact", P_override=None, sparse_s: int = 0):
        self.n, self.m, self.r = n, m, r
        self.W = np.array(W0, dtype=np.float64)
        self.M = np.zeros((r, m))
        self.V = np.zeros((r, m))
        self.state = LayerState(seed, layer_id, refresh_T)
        self.lr, self.beta1, self.beta2, self.eps, self.alpha = lr, beta1, beta2, eps, alpha
        self.mode = mode
        self.P_override = P_override      # explicit P for algebraic pins (orthonormal, identity)
        self.sparse_s = sparse_s          # > 0: sparse JL projection with this many terms per row

    def P(self, epoch: int | None = None) -> np.ndarray:
        if self.P_override is not None:
            return np.asarray(self.P_override, dtype=np.float64)
        ep = self.state.epoch if epoch is None else epoch
        return projection(self.state.seed, self.state.layer_id, ep, self.n, self.r, self.mode, self.sparse_s)

    def forward(self, X):
        return linear_fwd(X, self.W, self.P(), self.mode)

    def backward(self, dY, Z):
        return linear_bwd(dY, Z, self.W, self.mode)

    def backward_recompute(self, X, dY):
        return linear_bwd_recompute(X, dY, self.W, self.P(), self.mode)

    def update(self, Gc, lr: float | None = None) -> None:
        t = self.state.step + 1
        self.W, self.M, self.V = adam_update(
            self.W, Gc, self.M, self.V, t, self.P(), self.lr if lr is None else lr,
            self.beta1, self.beta2, self.eps, self.alpha, self.mode)
        self.state.advance()


def saved_elements(tokens: int, r: int) -> int:
    """Elements kept for backward per compressed linear (Table 1: b l n -> b l r)."""
    return tokens * r


def rel_frobenius(a, b) -> float:
    """||a - b||_F / ||b||_F with b the oracle's tensor."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    num = np.linalg.norm(a - b)
    return float(num / den) if den > 0 else float(num)
