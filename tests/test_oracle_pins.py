"""Pins for the CPU oracle: each checks it against something other than itself
(published vectors, closed forms, algebraic identities, library routines,
brute-force loops), chosen so a dropped term, wrong sign/index or transposed
operand fails at least one of them."""
import math
import os

import numpy as np
import pytest
import torch
from scipy import stats

from oracle import compact_oracle as co

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --- Philox integer stream vs published known-answer vectors ------------------
def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[:4], v[4:6], v[6:]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = co.philox4x32_10(np.array(ctr), np.array(key))
        assert [int(x) for x in got] == want


def test_philox_vectorised_equals_scalar_calls():
    ctr = np.array([[0, 0, 0, 0], [0xFFFFFFFF] * 4, [0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344]])
    key = np.array([[0, 0], [0xFFFFFFFF] * 2, [0xA4093822, 0x299F31D0]])
    got = co.philox4x32_10(ctr, key)
    for row, (_, _, want) in zip(got, _kat_rows()):
        assert [int(x) for x in row] == want


def test_projection_words_counter_layout():
    # word (i, 4q+w) is word w of philox(ctr=(q, i, layer, epoch), key=(seed_lo, seed_hi)); call q covers columns 8q .. 8q+7
    seed, layer, epoch = (0x1234 << 32) | 0x89ABCDEF, 5, 3
    words = co.projection_words(seed, layer, epoch, 9, 18)
    assert words.shape == (9, 12)
    for i, q in [(0, 0), (8, 2), (4, 1)]:
        ref = co.philox4x32_10(np.array([q, i, layer, epoch]), np.array([0x89ABCDEF, 0x1234]))
        assert (words[i, 4 * q:4 * q + 4] == ref).all()
    # the all-zero call is the first published vector
    w0 = co.projection_words(0, 0, 0, 1, 8)
    assert [int(x) for x in w0[0]] == _kat_rows()[0][2]
    # entry (i, j) comes from word (j >> 1) & 3 of call j >> 3: the cos of the word's pair for even j, the sin for odd j
    r = 18
    P = co.projection(seed, layer, epoch, 9, r) * math.sqrt(r)
    for i, j in [(0, 0), (3, 5), (8, 17), (4, 10)]:
        w = int(words[i, 4 * (j >> 3) + ((j >> 1) & 3)])
        rad = math.sqrt(-2 * math.log(((w & 0xFFFF) + 0.5) / 65536))
        ang = 2 * math.pi * (w >> 16) / 65536
        assert P[i, j] == pytest.approx(rad * (math.sin(ang) if j & 1 else math.cos(ang)), rel=1e-12, abs=1e-15)


# --- Box-Muller closed forms and distribution -----------------------------------
def test_box_muller_closed_forms():
    # a word's high half is the angle, its low half the radius
    lo = 0x8000
    rad = math.sqrt(-2 * math.log((lo + 0.5) / 65536))
    # u2 = 0 -> (rad, 0); u2 = 1/4 -> (0, rad); u2 = 1/2 -> (-rad, 0); u2 = 3/4 -> (0, -rad)
    w = np.array([[lo, (0x4000 << 16) | lo, (0x8000 << 16) | lo, (0xC000 << 16) | lo]], dtype=np.uint32)
    g = co.box_muller_from_words(w)[0]
    assert g.shape == (8,)
    assert g[0] == pytest.approx(rad, rel=1e-15) and g[1] == 0.0
    assert abs(g[2]) < 1e-15 and g[3] == pytest.approx(rad, rel=1e-15)
    assert g[4] == pytest.approx(-rad, rel=1e-15) and abs(g[5]) < 1e-15
    assert abs(g[6]) < 1e-15 and g[7] == pytest.approx(-rad, rel=1e-15)
    # extreme radii: u1 = 1 - 2^-17 and u1 = 2^-17
    w = np.array([[0x0000FFFF, 0x00000000]], dtype=np.uint32)
    g = co.box_muller_from_words(w)[0]
    assert g[0] == pytest.approx(math.sqrt(-2 * math.log1p(-2.0 ** -17)), rel=1e-9)
    assert g[0] == pytest.approx(3.9063e-3, rel=1e-4)
    assert g[2] == pytest.approx(math.sqrt(34 * math.log(2)), rel=1e-15)      # the largest radius: 4.8546
    assert g[2] == pytest.approx(4.8546, rel=1e-4)
    # the two halves do not leak into one another
    a = co.box_muller_from_words(np.array([[0x12345678]], dtype=np.uint32))[0]
    b = co.box_muller_from_words(np.array([[0x12340000 | 0x5678]], dtype=np.uint32))[0]
    assert np.array_equal(a, b)
    rad = math.sqrt(-2 * math.log((0x5678 + 0.5) / 65536))
    assert math.hypot(a[0], a[1]) == pytest.approx(rad, rel=1e-14)
    assert math.atan2(a[1], a[0]) == pytest.approx(2 * math.pi * 0x1234 / 65536, rel=1e-13)


def test_projection_distribution():
    r = 64
    P = co.projection(seed=7, layer_id=1, epoch=0, n=40000, r=r)
    x = (P * math.sqrt(r)).ravel()
    N = x.size
    assert abs(x.mean()) < 5 / math.sqrt(N)
    assert abs(x.var() - 1.0) < 5 * math.sqrt(2.0 / N)
    assert abs(stats.kurtosis(x, fisher=False) - 3.0) < 5 * math.sqrt(24.0 / N)
    assert abs(stats.skew(x)) < 5 * math.sqrt(6.0 / N)
    assert stats.kstest(x[:500000], "norm").pvalue > 1e-3
    # cos lanes and sin lanes are uncorrelated; columns are uncorrelated
    assert abs(np.corrcoef(P[:, 0], P[:, 1])[0, 1]) < 5 / math.sqrt(P.shape[0])
    assert abs(np.corrcoef(P[:, 1], P[:, 2])[0, 1]) < 5 / math.sqrt(P.shape[0])


def test_projection_scale_gives_identity():
    # E[P P^T] = I_n when the variance is 1/r (Section 3.3)
    n, r, S = 12, 8, 4000
    acc = np.zeros((n, n))
    for s in range(S):
        P = co.projection(seed=s, layer_id=0, epoch=0, n=n, r=r)
        acc += P @ P.T
    acc /= S
    d = np.diag(acc)
    off = acc - np.diag(d)
    assert np.all(np.abs(d - 1.0) < 5 * math.sqrt(2.0 / (r * S)))
    assert np.all(np.abs(off) < 5 * math.sqrt(1.0 / (r * S)))


def test_projection_depends_on_each_counter_word():
    base = co.projection(1, 2, 3, 6, 8)
    assert not np.array_equal(base, co.projection(2, 2, 3, 6, 8))
    assert not np.array_equal(base, co.projection(1 + (1 << 32), 2, 3, 6, 8))
    assert not np.array_equal(base, co.projection(1, 3, 3, 6, 8))
    assert not np.array_equal(base, co.projection(1, 2, 4, 6, 8))
    # a taller P with the same r shares the row prefix; ragged r is a column prefix
    assert np.array_equal(base, co.projection(1, 2, 3, 9, 8)[:6])
    assert np.allclose(co.projection(1, 2, 3, 6, 7) * math.sqrt(7), base[:, :7] * math.sqrt(8), rtol=1e-15)


# --- bf16 storage rounding --------------------------------------------------------
def _f32_from_bits(b):
    return float(np.array([b], dtype=np.uint32).view(np.float32)[0])


def test_round_bf16_bit_patterns():
    cases = {
        0x3F808000: 0x3F80,  # tie -> even (down)
        0x3F818000: 0x3F82,  # tie -> even (up)
        0x3F808001: 0x3F81,  # just above the tie
        0x3F807FFF: 0x3F80,
        0xBF818000: 0xBF82,
        0x00000000: 0x0000,
        0x00400000: 0x0040,  # bf16 subnormal kept
        0x00008000: 0x0000,  # half of the smallest subnormal: tie -> even (0)
        0x00018000: 0x0002,
        0x7F7FFFFF: 0x7F80,  # rounds up to +inf
    }
    for bits32, want16 in cases.items():
        y = co.round_bf16(np.array([_f32_from_bits(bits32)]))[0]
        got = int(np.array([y], dtype=np.float32).view(np.uint32)[0])
        assert got == want16 << 16, hex(bits32)
    assert np.isnan(co.round_bf16(np.array([np.nan]))[0])
    assert co.round_bf16(np.array([-np.inf]))[0] == -np.inf


def test_round_bf16_matches_torch_conversion():
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 2 ** 32, size=200000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float64).numpy()
    got = co.round_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)


# --- GEMM definitions: brute force on tiny shapes -------------------------------
def _brute_fwd(X, W, P):
    bl, n = len(X), len(W)
    m, r = len(W[0]), len(P[0])
    Y = [[sum(X[t][k] * W[k][c] for k in range(n)) for c in range(m)] for t in range(bl)]
    Z = [[sum(X[t][k] * P[k][j] for k in range(n)) for j in range(r)] for t in range(bl)]
    return Y, Z


def _brute_bwd(dY, Z, W):
    bl, m = len(dY), len(dY[0])
    n, r = len(W), len(Z[0])
    Gc = [[sum(Z[t][j] * dY[t][c] for t in range(bl)) for c in range(m)] for j in range(r)]
    dX = [[sum(dY[t][c] * W[k][c] for c in range(m)) for k in range(n)] for t in range(bl)]
    return dX, Gc


@pytest.mark.parametrize("bl,n,m,r", [(5, 7, 3, 4), (3, 6, 5, 5), (1, 2, 2, 1)])
def test_fwd_bwd_brute_force(bl, n, m, r):
    rng = np.random.default_rng(bl * 100 + r)
    X, W, dY = rng.standard_normal((bl, n)), rng.standard_normal((n, m)), rng.standard_normal((bl, m))
    P = co.projection(3, 1, 0, n, r)
    Y, Z = co.linear_fwd(X, W, P)
    Yb, Zb = _brute_fwd(X.tolist(), W.tolist(), P.tolist())
    assert np.allclose(Y, Yb, rtol=1e-13, atol=1e-13) and np.allclose(Z, Zb, rtol=1e-13, atol=1e-13)
    dX, Gc = co.linear_bwd(dY, Z, W)
    dXb, Gcb = _brute_bwd(dY.tolist(), Z.tolist(), W.tolist())
    assert np.allclose(dX, dXb, rtol=1e-13, atol=1e-13) and np.allclose(Gc, Gcb, rtol=1e-13, atol=1e-13)
    assert Y.shape == (bl, m) and Z.shape == (bl, r) and dX.shape == (bl, n) and Gc.shape == (r, m)


def test_update_brute_force():
    rng = np.random.default_rng(5)
    n, m, r = 4, 3, 2
    W, Gc = rng.standard_normal((n, m)), rng.standard_normal((r, m))
    M0, V0 = rng.standard_normal((r, m)), rng.random((r, m))
    P = co.projection(0, 0, 0, n, r)
    b1, b2, eps, lr, alpha, t = 0.8, 0.95, 1e-6, 0.01, 0.25, 3
    Wn, Mn, Vn = co.adam_update(W, Gc, M0, V0, t, P, lr, b1, b2, eps, alpha)
    for i in range(n):
        for c in range(m):
            acc = 0.0
            for j in range(r):
                mm = b1 * M0[j, c] + (1 - b1) * Gc[j, c]
                vv = b2 * V0[j, c] + (1 - b2) * Gc[j, c] ** 2
                assert Mn[j, c] == pytest.approx(mm, rel=1e-14)
                assert Vn[j, c] == pytest.approx(vv, rel=1e-14)
                nn = (mm / (1 - b1 ** t)) / (math.sqrt(vv / (1 - b2 ** t)) + eps)
                acc += P[i, j] * nn
            assert Wn[i, c] == pytest.approx(W[i, c] - lr * alpha * acc, rel=1e-13)


# --- Algebraic identities ----------------------------------------------------------
def test_compressed_gradient_is_projected_gradient():
    # (X P)^T dY = P^T (X^T dY): CompAct is GaLore with Q = I (Section 3.2)
    rng = np.random.default_rng(1)
    bl, n, m, r = 40, 24, 10, 6
    X, W, dY = rng.standard_normal((bl, n)), rng.standard_normal((n, m)), rng.standard_normal((bl, m))
    P = co.projection(11, 0, 0, n, r)
    _, Z = co.linear_fwd(X, W, P)
    _, Gc = co.linear_bwd(dY, Z, W)
    G = X.T @ dY
    assert np.allclose(Gc, P.T @ G, rtol=1e-12, atol=1e-12)


def test_orthonormal_full_rank_projection_recovers_gradient():
    # r = n and P orthonormal: P Gc = X^T dY exactly
    rng = np.random.default_rng(2)
    bl, n, m = 30, 16, 9
    X, W, dY = rng.standard_normal((bl, n)), rng.standard_normal((n, m)), rng.standard_normal((bl, m))
    Q, _ = np.linalg.qr(co.projection(4, 0, 0, n, n))
    _, Z = co.linear_fwd(X, W, Q)
    _, Gc = co.linear_bwd(dY, Z, W)
    assert np.allclose(Q @ Gc, X.T @ dY, rtol=1e-12, atol=1e-12)


def test_dx_is_gradient_of_inner_product():
    # d/dX <X W, dY> = dY W^T : finite difference on one entry
    rng = np.random.default_rng(3)
    X, W, dY = rng.standard_normal((4, 5)), rng.standard_normal((5, 3)), rng.standard_normal((4, 3))
    P = co.projection(0, 0, 0, 5, 2)
    dX, _ = co.linear_bwd(dY, co.linear_fwd(X, W, P)[1], W)
    h = 1e-6
    for (t, k) in [(0, 0), (3, 4), (2, 1)]:
        Xp = X.copy(); Xp[t, k] += h
        Xm = X.copy(); Xm[t, k] -= h
        fd = (np.sum(co.linear_fwd(Xp, W, P)[0] * dY) - np.sum(co.linear_fwd(Xm, W, P)[0] * dY)) / (2 * h)
        assert dX[t, k] == pytest.approx(fd, rel=1e-7)


def test_bwd_recompute_is_the_sketched_gradient_by_brute_force():
    # without a stored z the compressed gradient is still P^T (X^T dY): element loops on a tiny case,
    # and with r = n and an orthonormal P the full gradient comes back
    rng = np.random.default_rng(8)
    bl, n, m, r = 7, 6, 5, 3
    X, W, dY = rng.standard_normal((bl, n)), rng.standard_normal((n, m)), rng.standard_normal((bl, m))
    P = co.projection(11, 2, 1, n, r)
    dX, Gc = co.linear_bwd_recompute(X, dY, W, P)
    for j in range(r):
        for c in range(m):
            want = sum(P[i, j] * X[t, i] * dY[t, c] for t in range(bl) for i in range(n))
            assert Gc[j, c] == pytest.approx(want, rel=1e-12, abs=1e-13)
    for t in range(bl):
        for i in range(n):
            assert dX[t, i] == pytest.approx(sum(dY[t, c] * W[i, c] for c in range(m)), rel=1e-12, abs=1e-13)
    Q, _ = np.linalg.qr(co.projection(4, 0, 0, n, n))
    _, Gq = co.linear_bwd_recompute(X, dY, W, Q)
    assert np.allclose(Q @ Gq, X.T @ dY, rtol=1e-12, atol=1e-12)
    # bf16 storage: z is rounded where Algorithm 1 would have stored it
    _, Gb = co.linear_bwd_recompute(X, dY, W, P, mode="bf16")
    assert np.array_equal(Gb, co.linear_bwd(dY, co.round_bf16(X @ P), W, mode="bf16")[1])


def test_group_backward_is_gradient_of_summed_inner_products():
    # layers sharing x: d/dx sum_g <x W_g, dY_g> by finite differences, Gc_g by element loops
    rng = np.random.default_rng(9)
    bl, n = 5, 6
    ms, rs = [4, 3, 4], [2, 3, 2]
    X = rng.standard_normal((bl, n))
    Ws = [rng.standard_normal((n, m)) for m in ms]
    dYs = [rng.standard_normal((bl, m)) for m in ms]
    Ps = [co.projection(21, g, 0, n, r) for g, r in enumerate(rs)]
    Ys, Zs = co.group_fwd(X, Ws, Ps)
    for g in range(3):
        assert np.allclose(Ys[g], X @ Ws[g], rtol=1e-13) and np.allclose(Zs[g], X @ Ps[g], rtol=1e-13)
    dX, Gcs = co.group_bwd(dYs, Zs, Ws)
    f = lambda x: sum(np.sum((x @ W) * dY) for W, dY in zip(Ws, dYs))
    h = 1e-6
    for (t, k) in [(0, 0), (4, 5), (2, 3)]:
        Xp = X.copy(); Xp[t, k] += h
        Xm = X.copy(); Xm[t, k] -= h
        assert dX[t, k] == pytest.approx((f(Xp) - f(Xm)) / (2 * h), rel=1e-7)
    for g in range(3):
        for j in range(rs[g]):
            for c in range(ms[g]):
                want = sum(Zs[g][t, j] * dYs[g][t, c] for t in range(bl))
                assert Gcs[g][j, c] == pytest.approx(want, rel=1e-12, abs=1e-13)
    # a group of one is the single layer
    d1, g1 = co.group_bwd(dYs[:1], Zs[:1], Ws[:1])
    d2, g2 = co.linear_bwd(dYs[0], Zs[0], Ws[0])
    assert np.array_equal(d1, d2) and np.array_equal(g1[0], g2)


# --- Adam ----------------------------------------------------------------------------
def test_adam_constant_gradient_closed_form():
    rng = np.random.default_rng(4)
    n, m, r, k = 10, 6, 4, 7
    g = rng.standard_normal((r, m))
    W0 = rng.standard_normal((n, m))
    lr, alpha, eps = 3e-3, 0.25, 1e-8
    lay = co.CompActLayerOracle(W0, n, m, r, seed=9, layer_id=2, refresh_T=0, lr=lr,
                                beta1=0.7, beta2=0.93, eps=eps, alpha=alpha)
    for _ in range(k):
        lay.update(g)
    N = g / (np.abs(g) + eps)
    want = W0 - k * lr * alpha * (lay.P() @ N)
    assert np.allclose(lay.W, want, rtol=1e-12, atol=1e-12)


def test_adam_identity_projection_equals_torch_adam():
    # r = n, P = I, alpha = 1: CompAct is plain Adam on W with gradient X^T dY
    rng = np.random.default_rng(6)
    bl, n, m, steps = 12, 5, 4, 5
    W0 = rng.standard_normal((n, m))
    lay = co.CompActLayerOracle(W0, n, m, n, seed=0, layer_id=0, refresh_T=2, lr=1e-2,
                                beta1=0.9, beta2=0.999, eps=1e-8, P_override=np.eye(n))
    Wt = torch.tensor(W0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([Wt], lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.0)
    for s in range(steps):
        X, dY = rng.standard_normal((bl, n)), rng.standard_normal((bl, m))
        Y, Z = lay.forward(X)
        _, Gc = lay.backward(dY, Z)
        lay.update(Gc)
        opt.zero_grad()
        Wt.grad = torch.tensor(X.T @ dY)
        opt.step()
        assert np.allclose(lay.W, Wt.detach().numpy(), rtol=1e-10, atol=1e-12), s
    assert lay.state.step == steps


def test_zero_inputs_change_nothing():
    rng = np.random.default_rng(8)
    n, m, r, bl = 6, 5, 3, 4
    W0 = rng.standard_normal((n, m))
    lay = co.CompActLayerOracle(W0, n, m, r, 1, 0, 0, 1e-2, 0.9, 0.999, 1e-8)
    Y, Z = lay.forward(np.zeros((bl, n)))
    assert not Y.any() and not Z.any()
    dX, Gc = lay.backward(rng.standard_normal((bl, m)), Z)
    assert not Gc.any()
    lay.update(Gc)
    assert np.array_equal(lay.W, W0) and not lay.M.any() and not lay.V.any()
    dX, Gc = lay.backward(np.zeros((bl, m)), rng.standard_normal((bl, r)))
    assert not dX.any() and not Gc.any()


# --- Refresh schedule (Algorithm 3 lines 10-13) -------------------------------------
def test_refresh_schedule():
    st = co.LayerState(seed=0, layer_id=0, refresh_T=2)
    used = []
    for _ in range(3):
        used.append(st.epoch)
        st.advance()
    assert used == [0, 0, 1] and st.epoch == 1 and st.step == 3
    st = co.LayerState(seed=0, layer_id=0, refresh_T=0)
    for _ in range(10):
        st.advance()
    assert st.epoch == 0
    st = co.LayerState(seed=0, layer_id=0, refresh_T=10)
    eps = []
    for _ in range(20):
        eps.append(st.epoch)
        st.advance()
    assert eps == [0] * 10 + [1] * 10 and st.epoch == 2
    assert not np.array_equal(co.projection(0, 0, 0, 8, 4), co.projection(0, 0, 1, 8, 4))


def test_layer_uses_refreshed_projection():
    rng = np.random.default_rng(10)
    n, m, r = 6, 4, 2
    lay = co.CompActLayerOracle(rng.standard_normal((n, m)), n, m, r, 5, 1, 1, 1e-2, 0.9, 0.999, 1e-8)
    P0 = lay.P()
    lay.update(rng.standard_normal((r, m)))
    assert lay.state.epoch == 1
    assert np.array_equal(lay.P(), co.projection(5, 1, 1, n, r)) and not np.array_equal(lay.P(), P0)


# --- bf16 storage mode: rounding happens at the stated points only --------------------
def test_bf16_mode_rounding_points():
    rng = np.random.default_rng(12)
    bl, n, m, r = 9, 8, 6, 4
    rb = co.round_bf16
    X, W, dY = rb(rng.standard_normal((bl, n))), rb(rng.standard_normal((n, m))), rb(rng.standard_normal((bl, m)))
    P = co.projection(2, 0, 0, n, r, mode="bf16")
    assert np.array_equal(P, rb(co.projection(2, 0, 0, n, r)))
    Y, Z = co.linear_fwd(X, W, P, mode="bf16")
    assert np.array_equal(Y, rb(X @ W)) and np.array_equal(Z, rb(X @ P))
    dX, Gc = co.linear_bwd(dY, Z, W, mode="bf16")
    assert np.array_equal(dX, rb(dY @ W.T)) and np.array_equal(Gc, Z.T @ dY)
    Wn, Mn, Vn = co.adam_update(W, Gc, np.zeros((r, m)), np.zeros((r, m)), 1, P, 1e-3, 0.9, 0.999, 1e-8, mode="bf16")
    N = rb((0.1 * Gc / 0.1) / (np.sqrt(0.001 * Gc * Gc / 0.001) + 1e-8))
    assert np.allclose(Wn, rb(W - 1e-3 * (P @ N)), rtol=0, atol=1e-2 * np.abs(W).max() * 2 ** -8)
    assert np.array_equal(Wn, rb(Wn))


# --- Memory accounting (Table 1, Table 3 with Appendix E) ----------------------------
def test_saved_activation_accounting():
    bl = 64 * 256
    assert co.saved_elements(bl, 256) == bl * 256
    n, m = 1024, 2736
    dense = bl * (2 * n + m)                         # x2 (shared by q,k,v), x6 (gate, up), x7 (down)
    comp = 3 * co.saved_elements(bl, n // 4) + 2 * co.saved_elements(bl, n // 4) + co.saved_elements(bl, m // 4)
    assert comp / dense == pytest.approx(1964 / 4784)
    assert 7.0 * comp / dense == pytest.approx(2.87, abs=0.005)   # Table 3 activation row at r = n/4


# --- The yardstick itself: relative Frobenius error, whole tensors and tiles -------------
def test_rel_frobenius_hand_values():
    b = np.array([[3.0, 0.0], [0.0, 4.0]])                      # ||b|| = 5
    a = b + np.array([[0.0, 0.3], [0.4, 0.0]])                  # ||a - b|| = 0.5
    assert co.rel_frobenius(a, b) == pytest.approx(0.1, rel=1e-12)
    assert co.rel_frobenius(b, b) == 0.0
    assert co.rel_frobenius(2 * b, b) == pytest.approx(1.0)     # not symmetric: measured against the second argument
    assert co.rel_frobenius(b, 2 * b) == pytest.approx(0.5)
    # zero oracle tensor: the absolute norm of the difference
    assert co.rel_frobenius(np.array([3.0, 4.0]), np.zeros(2)) == pytest.approx(5.0)
    assert co.rel_frobenius(np.zeros((2, 3)), np.zeros((2, 3))) == 0.0
    # a 1-D sum written out
    x, y = np.array([1.0, 2.0, 2.0]), np.array([2.0, 2.0, 1.0])
    assert co.rel_frobenius(x, y) == pytest.approx(math.sqrt(2.0) / 3.0)


def test_tile_metric_hand_values():
    from tests._harness import tile_sq_norms, worst_tile
    a = np.arange(12, dtype=np.float64).reshape(3, 4)            # tiles of 2 x 3: ragged on both edges
    want = np.array([[0 + 1 + 4 + 16 + 25 + 36, 9 + 49], [64 + 81 + 100, 121]], dtype=np.float64)
    assert np.array_equal(tile_sq_norms(a, 2, 3), want)
    b = np.ones((4, 4))
    e = np.zeros((4, 4))
    e[3, 3] = 0.2                                                # one wrong entry in the last 2 x 2 tile
    assert worst_tile(b + e, b, (2, 2)) == pytest.approx(0.1)    # 0.2 / ||ones(2,2)||
    assert co.rel_frobenius(b + e, b) == pytest.approx(0.05)     # the whole-tensor figure blurs it
    assert worst_tile(b, b, (2, 2)) == 0.0
    # a wrong tile of a large tensor passes the whole-tensor bound and fails the tile bound
    rng = np.random.default_rng(0)
    big = rng.standard_normal((1024, 512))
    bad = big.copy()
    bad[128:256, 64:128] = 0.0
    assert co.rel_frobenius(bad, big) < 0.2 and worst_tile(bad, big, (128, 64)) == pytest.approx(1.0)


# --- Sparse Johnson-Lindenstrauss projection (Ablation Study) ------------------------------------
def test_sparse_jl_terms_counter_layout_and_hash():
    seed, layer, epoch, n, r, s = (7 << 32) | 99, 3, 2, 5, 37, 6
    cols, signs = co.sparse_jl_terms(seed, layer, epoch, n, r, s)
    assert cols.shape == signs.shape == (n, s)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i in range(n):
        for t in range(s):
            w = int(co.philox4x32_10([0x80000000 | (t >> 2), i, layer, epoch], key)[t & 3])   # pinned by the KATs
            assert cols[i, t] == ((w & 0x7FFFFFFF) * r) >> 31 and signs[i, t] == (-1 if w >> 31 else 1)
    assert cols.min() >= 0 and cols.max() < r
    # the stream is its own: word 0 of the counter has its top bit set, so no call coincides with one behind the
    # Gaussian projection of the same layer (whose word 0 is a column group below 2^30)
    g = co.projection_words(seed, layer, epoch, n, 8)
    first = np.array([int(co.philox4x32_10([0x80000000, i, layer, epoch], key)[0]) for i in range(n)])
    assert not np.any(first == g[:, 0])


def test_sparse_jl_projection_structure():
    n, r, s = 300, 64, 8
    P = co.projection_sparse_jl(5, 1, 0, n, r, s)
    K = P * math.sqrt(s)
    assert np.array_equal(K, np.rint(K))                                   # integer counts times 1/sqrt(s)
    per_row = np.abs(K).sum(axis=1)
    assert np.all(per_row <= s) and np.all((s - per_row) % 2 == 0)          # terms that cancel go in pairs
    cols, signs = co.sparse_jl_terms(5, 1, 0, n, r, s)
    distinct = np.array([len(set(c)) == s for c in cols])
    assert distinct.any() and np.all(np.count_nonzero(K[distinct], axis=1) == s)   # no collision: exactly s entries of +-1
    assert np.all(np.abs(K[distinct]).max(axis=1) == 1)
    # a hand-built row: terms (col 2, +), (col 2, +), (col 0, -) give counts [-1, 0, 2]
    Kh = np.zeros(3)
    for c, sg in ((2, 1), (2, 1), (0, -1)):
        Kh[c] += sg
    assert list(Kh) == [-1.0, 0.0, 2.0]
    # other epoch, layer or seed: another matrix; through the generic entry point: the same one
    assert not np.array_equal(P, co.projection_sparse_jl(5, 1, 1, n, r, s))
    assert not np.array_equal(P, co.projection_sparse_jl(5, 2, 0, n, r, s))
    assert np.array_equal(P, co.projection(5, 1, 0, n, r, mode="bf16", sparse_s=s))


def test_sparse_jl_scale_gives_identity_and_uniform_columns():
    n, r, s, S = 6, 16, 4, 6000
    acc = np.zeros((n, n))
    for seed in range(S):
        P = co.projection_sparse_jl(seed, 0, 0, n, r, s)
        acc += P @ P.T
    acc /= S
    # diagonal: (1/s) * sum_j (count_j)^2 has mean 1; off-diagonal: mean 0, variance 1/r
    assert np.all(np.abs(np.diag(acc) - 1.0) < 5 * math.sqrt(2.0 / (r * S)) + 5e-3)
    off = acc - np.diag(np.diag(acc))
    assert np.all(np.abs(off) < 5 * math.sqrt(1.0 / (r * S)))
    cols, signs = co.sparse_jl_terms(1, 0, 0, 20000, 50, 8)
    counts = np.bincount(cols.ravel(), minlength=50)
    assert stats.chisquare(counts).pvalue > 1e-4
    assert abs(signs.mean()) < 5 / math.sqrt(signs.size)


def test_sparse_jl_layer_steps_like_the_dense_one():
    # the layer with a sparse projection is Algorithms 1-3 with that P: compare with element loops
    rng = np.random.default_rng(21)
    bl, n, m, r, s = 5, 7, 4, 3, 2
    lay = co.CompActLayerOracle(rng.standard_normal((n, m)), n, m, r, 9, 2, 0, 1e-2, 0.9, 0.999, 1e-8, sparse_s=s)
    P = co.projection_sparse_jl(9, 2, 0, n, r, s)
    assert np.array_equal(lay.P(), P)
    X, dY = rng.standard_normal((bl, n)), rng.standard_normal((bl, m))
    Y, Z = lay.forward(X)
    Zl = np.zeros((bl, r))
    cols, signs = co.sparse_jl_terms(9, 2, 0, n, r, s)
    for t in range(bl):
        for i in range(n):
            for k in range(s):
                Zl[t, cols[i, k]] += signs[i, k] * X[t, i] / math.sqrt(s)       # the signed gather the construction describes
    assert np.allclose(Z, Zl, rtol=0, atol=1e-12)
    W0 = lay.W.copy()
    _, Gc = lay.backward(dY, Z)
    lay.update(Gc)
    N = (0.1 * Gc / 0.1) / (np.sqrt(0.001 * Gc * Gc / 0.001) + 1e-8)
    Wl = W0.copy()
    for i in range(n):
        for k in range(s):
            Wl[i] -= 1e-2 * signs[i, k] * N[cols[i, k]] / math.sqrt(s)          # the signed scatter of rows of N
    assert np.allclose(lay.W, Wl, rtol=0, atol=1e-12)
