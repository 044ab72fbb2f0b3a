"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these compares the oracle with itself: each expected value comes from a
closed form, from a library routine (scipy softmax, torch SDPA), from an
independent brute-force restatement (pairwise kernel form of Eq. 4/9, Python
sets for the three memories), or from an invariant of the method.
"""
import numpy as np
import pytest
import scipy.special
from hypothesis import given, settings, strategies as st

from oracle.lola_oracle import (LolaOracle, OracleConfig, UnitState, phi, round_bf16, sre_scores)

RNG = np.random.default_rng(20250523)


def lib_phi(x, W, kind="softmax"):
    """Feature map built from library routines only (independent of oracle.phi)."""
    u = np.einsum("nd,df->nf", x, W)
    if kind == "exp":
        return np.concatenate([np.exp(u), 1.0 / np.exp(u)], axis=1)
    return np.concatenate([scipy.special.softmax(u, axis=1), scipy.special.softmax(-u, axis=1)], axis=1)


def nearest_bf16(x):
    """Nearest value with 8 significant bits (ties to even) of float64 data, by scaling to integers: an
    independent statement of the rounding (a cast through float32 would round twice)."""
    x = np.asarray(x, dtype=np.float64)
    e = np.floor(np.log2(np.abs(np.where(x == 0, 1.0, x))))
    ulp = 2.0 ** (e - 7)
    return np.where(x == 0, 0.0, np.rint(x / ulp) * ulp)


def make_unit(d=8, F=4, eta=4, lam=3, kind="softmax", rounding="none", schedule="eager", rng=RNG):
    cfg = OracleConfig(1, 1, 1, d, F, eta, lam, phi_kind=kind, operand_rounding=rounding, schedule=schedule)
    W = rng.standard_normal((d, F)) / np.sqrt(d)
    return UnitState(cfg, W), cfg, W


def rand_qkv(n, d, g=1, rng=RNG, clustered=True):
    q = rng.standard_normal((g, n, d))
    if clustered:
        mu = rng.standard_normal((4, d))
        k = mu[rng.integers(0, 4, n)] + 0.3 * rng.standard_normal((n, d))
    else:
        k = rng.standard_normal((n, d))
    v = rng.standard_normal((n, d))
    return q, k, v


# ------------------------------------------------------------------ feature map (Eq. 6 / softmax halves)
def test_phi_matches_library_softmax_and_exp():
    x = RNG.standard_normal((7, 16))
    W = RNG.standard_normal((16, 5))
    f = phi(x, W, "softmax")
    assert f.shape == (7, 10)
    np.testing.assert_allclose(f, lib_phi(x, W, "softmax"), rtol=1e-13, atol=0)
    np.testing.assert_allclose(f[:, :5].sum(1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(f[:, 5:].sum(1), 1.0, rtol=1e-13)
    assert (f > 0).all()
    e = phi(x, W, "exp")
    # Eq. 6: second half is the reciprocal of the first, entry by entry, and entry i is exp(w_i . x)
    np.testing.assert_allclose(e[:, :5] * e[:, 5:], 1.0, rtol=1e-12)
    i, j = 3, 2
    np.testing.assert_allclose(e[i, j], np.exp(sum(W[a, j] * x[i, a] for a in range(16))), rtol=1e-12)


def test_phi_transposed_operand_would_fail():
    # W is [d, F] with d != F: the first half must respond to column f of W, not row f
    d, F = 6, 3
    W = np.zeros((d, F))
    W[0, 2] = 5.0
    x = np.zeros((1, d))
    x[0, 0] = 1.0
    f = phi(x, W, "softmax")[0]
    assert np.argmax(f[:F]) == 2 and np.argmin(f[F:]) == 2


def test_round_bf16_grid_and_ties():
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: ties to even -> 1; 1 + 3*2^-8 -> 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, -0.3, 3.14159, 1e-40, 0.0])
    r = round_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2.0 ** -6 and r[3] == 1.0 + 2.0 ** -7
    import torch
    ref = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(r, ref)
    y = RNG.standard_normal(5000) * np.exp(RNG.uniform(-20, 20, 5000))
    ref = torch.tensor(y, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(round_bf16(y), ref)


# ------------------------------------------------------------------ I4: self-recall error (Eq. 9, 10)
def test_sre_zero_for_exactly_stored_pair():
    d, F = 8, 4
    W = RNG.standard_normal((d, F))
    k = RNG.standard_normal((1, d))
    v = RNG.standard_normal((1, d))
    f = lib_phi(k, W)
    H = f.T @ v
    s = f[0]
    assert sre_scores(phi(k, W), v, H, s)[0] < 1e-14


def test_sre_shared_key_closed_form():
    # n pairs with one key: the hidden state recalls the mean value, SRE_i = ||v_i - mean v||
    d, F, n = 8, 4, 6
    W = RNG.standard_normal((d, F))
    k = np.repeat(RNG.standard_normal((1, d)), n, axis=0)
    v = RNG.standard_normal((n, d))
    f = lib_phi(k, W)
    H = f.T @ v
    s = f.sum(0)
    want = np.linalg.norm(v - v.mean(0, keepdims=True), axis=1)
    np.testing.assert_allclose(sre_scores(phi(k, W), v, H, s), want, rtol=1e-12)


def test_sre_is_norm_not_squared_and_zero_state_gives_norm_v():
    d, F = 8, 4
    W = RNG.standard_normal((d, F))
    k = RNG.standard_normal((3, d))
    v = RNG.standard_normal((3, d))
    sc = sre_scores(phi(k, W), v, np.zeros((2 * F, d)), np.zeros(2 * F))
    np.testing.assert_allclose(sc, np.sqrt((v * v).sum(1)), rtol=1e-14)


def test_sre_pairwise_kernel_form():
    # Eq. 9 written pair by pair: m(k) = sum_j (phi(k).phi(k_j)) v_j / sum_j phi(k).phi(k_j)
    d, F, n = 6, 3, 9
    W = RNG.standard_normal((d, F))
    ks, vs = RNG.standard_normal((n, d)), RNG.standard_normal((n, d))
    kq, vq = RNG.standard_normal((4, d)), RNG.standard_normal((4, d))
    fk, fq = lib_phi(ks, W, "exp"), lib_phi(kq, W, "exp")
    H, s = fk.T @ vs, fk.sum(0)
    want = []
    for i in range(4):
        w = np.array([fq[i] @ fk[j] for j in range(n)])
        want.append(np.linalg.norm((w[:, None] * vs).sum(0) / w.sum() - vq[i]))
    np.testing.assert_allclose(sre_scores(phi(kq, W, "exp"), vq, H, s), want, rtol=1e-12)


# ------------------------------------------------------------------ I1: decode, eta = 0, lambda = 0
@pytest.mark.parametrize("kind", ["softmax", "exp"])
def test_decode_no_window_no_cache_is_causal_linear_attention(kind):
    d, F, n, g = 8, 4, 20, 2
    u, cfg, W = make_unit(d, F, eta=0, lam=0, kind=kind)
    q, k, v = rand_qkv(n, d, g)
    if kind == "exp":
        q, k = 0.3 * q, 0.3 * k
    fk = lib_phi(k, W, kind)
    for t in range(n):
        out = u.decode_step(q[:, t], k[t], v[t])
        fq = lib_phi(q[:, t], W, kind)
        for h in range(g):
            num = sum((fq[h] @ fk[j]) * v[j] for j in range(t + 1))      # Eq. 4, brute force
            den = sum(fq[h] @ fk[j] for j in range(t + 1))
            np.testing.assert_allclose(out[h], num / den, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ I2: lambda = 0 closed form (prefill)
@pytest.mark.parametrize("eta,C", [(4, 4), (8, 4), (3, 5), (0, 4), (4, 1)])
def test_prefill_without_sparse_cache_closed_form(eta, C):
    d, F, n, g = 8, 4, 23, 2
    u, cfg, W = make_unit(d, F, eta=eta, lam=0)
    q, k, v = rand_qkv(n, d, g)
    fk = lib_phi(k, W)
    scale = 1.0 / np.sqrt(d)
    t0 = 0
    while t0 < n:
        c = min(C, n - t0)
        out = u.prefill_chunk(q[:, t0:t0 + c], k[t0:t0 + c], v[t0:t0 + c])
        w0 = max(0, t0 - eta)                       # first position still held with softmax
        for r in range(c):
            t = t0 + r
            for h in range(g):
                fq = lib_phi(q[h, t:t + 1], W)[0]
                num = np.zeros(d)
                den = 0.0
                for j in range(0, w0):              # linear part: everything older than the window
                    num += (fq @ fk[j]) * v[j]
                    den += fq @ fk[j]
                for j in range(w0, t + 1):          # softmax part: window + causal chunk
                    e = np.exp(q[h, t] @ k[j] * scale)
                    num += e * v[j]
                    den += e
                np.testing.assert_allclose(out[h, r], num / den, rtol=1e-10, atol=1e-12)
        t0 += c


# ------------------------------------------------------------------ I3: caches large enough => softmax attention
@pytest.mark.parametrize("eta,lam,C", [(8, 64, 8), (64, 0, 16), (4, 60, 4), (0, 64, 8)])
def test_large_cache_equals_causal_softmax_attention(eta, lam, C):
    import torch
    B, Hq, Hkv, d, F, n = 2, 4, 2, 16, 4, 64
    cfg = OracleConfig(B, Hq, Hkv, d, F, eta, lam)
    W = RNG.standard_normal((Hkv, d, F))
    orc = LolaOracle(cfg, W)
    q = RNG.standard_normal((B, n, Hq, d))
    k = RNG.standard_normal((B, n, Hkv, d))
    v = RNG.standard_normal((B, n, Hkv, d))
    outs = [orc.prefill_chunk(q[:, t:t + C], k[:, t:t + C], v[:, t:t + C]) for t in range(0, n, C)]
    out = np.concatenate(outs, axis=1)
    tq = torch.tensor(q).permute(0, 2, 1, 3)
    tk = torch.tensor(k).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    tv = torch.tensor(v).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
    st_ = orc.read_state()
    assert np.all(st_["H"] == 0) and np.all(st_["s"] == 0)
    assert all(u.n_scored_updates == 0 for row in orc.units for u in row)


def test_decode_large_cache_equals_softmax_attention():
    import torch
    d, F, n, g = 16, 4, 40, 2
    u, cfg, W = make_unit(d, F, eta=5, lam=64)
    q, k, v = rand_qkv(n, d, g)
    for t in range(n):
        out = u.decode_step(q[:, t], k[t], v[t])
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(q[:, t:t + 1]), torch.tensor(k[None, :t + 1]).expand(g, -1, -1),
            torch.tensor(v[None, :t + 1]).expand(g, -1, -1)).numpy()[:, 0]
        np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
    assert np.all(u.H == 0)


# ------------------------------------------------------------------ I5 / I6: conservation and selection
def run_unit(u, q, k, v, C, decode_tail=0):
    n = k.shape[0]
    outs = []
    t = 0
    while t < n - decode_tail:
        c = min(C, n - decode_tail - t)
        outs.append(u.prefill_chunk(q[:, t:t + c], k[t:t + c], v[t:t + c]))
        t += c
    for t in range(n - decode_tail, n):
        outs.append(u.decode_step(q[:, t], k[t], v[t])[:, None])
    return np.concatenate(outs, axis=1)


@pytest.mark.parametrize("rounding", ["none", "bf16"])
@pytest.mark.parametrize("eta,lam,C,tail", [(8, 6, 8, 0), (8, 6, 4, 5), (5, 9, 3, 0), (0, 4, 4, 3), (8, 1, 8, 8)])
def test_conservation_and_selection(eta, lam, C, tail, rounding):
    d, F, n = 8, 4, 61
    u, cfg, W = make_unit(d, F, eta=eta, lam=lam, rounding=rounding)
    q, k, v = rand_qkv(n, d, 1)
    seen_folded = set()
    t = 0
    steps = [("p", min(C, n - tail - t0)) for t0 in range(0, n - tail, C)] + [("d", 1)] * tail
    for kind_, c in steps:
        H0, s0 = u.H.copy(), u.s.copy()
        if kind_ == "p":
            u.prefill_chunk(q[:, t:t + c], k[t:t + c], v[t:t + c])
        else:
            u.decode_step(q[:, t], k[t], v[t])
        t += c
        win, G, fold = set(map(int, u.win_pos)), set(map(int, u.G_pos)), set(u.folded_pos)
        # every past pair is in exactly one memory
        assert len(u.folded_pos) == len(fold)
        assert not (win & G) and not (win & fold) and not (G & fold)
        assert win | G | fold == set(range(t))
        assert win == set(range(max(0, t - eta), t))
        # folded pairs never come back
        assert seen_folded <= fold
        newly = fold - seen_folded
        seen_folded = set(fold)
        # |G| = min(lambda, number of pairs that ever left the window)
        assert len(G) == min(lam, t - len(win))
        # cached pairs are exact copies
        for i, p in enumerate(u.G_pos):
            assert np.array_equal(u.G_k[i], k[p]) and np.array_equal(u.G_v[i], v[p])
        # H, s are the sum over folded pairs, from scratch
        # (Eq. 13 folds phi(k) itself in both variants; the "bf16" variant rounds operands of Eq. 10 only)
        f = lib_phi(k[sorted(fold)], W) if fold else np.zeros((0, 2 * F))
        np.testing.assert_allclose(u.H, f.T @ v[sorted(fold)] if fold else 0 * u.H, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(u.s, f.sum(0) if fold else 0 * u.s, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(u.s.sum(), 2.0 * len(fold), rtol=1e-10)
        # the selection equals a full sort of the eligible set scored against the state before the fold
        if newly and lam > 0:
            E = sorted(G | newly)
            fE = lib_phi(k[E], W)
            H0r = H0
            if rounding == "bf16":
                fE, H0r = nearest_bf16(fE), nearest_bf16(H0)
            den = fE @ s0
            vh = np.where(den[:, None] > 0, (fE @ H0r) / np.where(den > 0, den, 1.0)[:, None], 0.0)
            sc = np.linalg.norm(vh - v[E], axis=1)
            ranked = sorted(range(len(E)), key=lambda i: (-sc[i], E[i]))
            assert set(E[i] for i in ranked[:lam]) == G
            assert min(sc[i] for i in ranked[:lam]) >= max(sc[i] for i in ranked[lam:])
            np.testing.assert_allclose(u.last_kept_min, min(sc[i] for i in ranked[:lam]), rtol=1e-9)
            np.testing.assert_allclose(u.last_folded_max, max(sc[i] for i in ranked[lam:]), rtol=1e-9)


def test_ties_keep_the_older_pair():
    # identical pairs => identical scores: the newer ones fold
    d, F = 8, 4
    u, cfg, W = make_unit(d, F, eta=2, lam=2)
    k1, v1 = RNG.standard_normal(d), RNG.standard_normal(d)
    n = 8
    k = np.repeat(k1[None], n, 0)
    v = np.repeat(v1[None], n, 0)
    q = RNG.standard_normal((1, n, d))
    run_unit(u, q, k, v, C=2)
    assert sorted(map(int, u.G_pos)) == [0, 1]
    assert sorted(u.folded_pos) == [2, 3, 4, 5]


# ------------------------------------------------------------------ I7: independence, slot order, stabiliser
def test_units_are_independent_and_slot_order_is_irrelevant():
    B, Hq, Hkv, d, F, n, C = 2, 4, 2, 8, 4, 48, 8
    cfg = OracleConfig(B, Hq, Hkv, d, F, 8, 5)
    W = RNG.standard_normal((Hkv, d, F))
    q = RNG.standard_normal((B, n, Hq, d))
    k = RNG.standard_normal((B, n, Hkv, d))
    v = RNG.standard_normal((B, n, Hkv, d))
    full = LolaOracle(cfg, W)
    out = np.concatenate([full.prefill_chunk(q[:, t:t + C], k[:, t:t + C], v[:, t:t + C]) for t in range(0, n, C)], 1)
    # one unit alone (batch row 1, KV head 1), with its sparse-cache slots shuffled before every call
    solo = UnitState(OracleConfig(1, 2, 1, d, F, 8, 5), W[1])
    outs = []
    for t in range(0, n, C):
        perm = RNG.permutation(len(solo.G_pos))
        solo.G_pos, solo.G_k, solo.G_v, solo.G_score = solo.G_pos[perm], solo.G_k[perm], solo.G_v[perm], solo.G_score[perm]
        outs.append(solo.prefill_chunk(q[1, t:t + C, 2:4].transpose(1, 0, 2), k[1, t:t + C, 1], v[1, t:t + C, 1]))
    np.testing.assert_allclose(np.concatenate(outs, 1).transpose(1, 0, 2), out[1, :, 2:4], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(solo.H, full.units[1][1].H, rtol=1e-12, atol=1e-14)


def test_output_is_eq14_without_stabiliser():
    # Eq. 14 literally, raw exponentials, from the oracle's own memories after some updates
    d, F, n, C = 8, 4, 40, 4
    u, cfg, W = make_unit(d, F, eta=4, lam=5)
    q, k, v = rand_qkv(n, d, 1)
    run_unit(u, q, k, v, C)
    qt = RNG.standard_normal((1, d)) * 3.0
    kt, vt = RNG.standard_normal(d), RNG.standard_normal(d)
    H, s = u.H.copy(), u.s.copy()
    out = u.decode_step(qt, kt, vt)[0]
    # after the update: G_t, window (new pair included), H_t, s_t
    fq = lib_phi(qt, W)[0]
    num = fq @ u.H
    den = fq @ u.s
    for kk, vv in list(zip(u.G_k, u.G_v)) + list(zip(u.win_k, u.win_v)):
        e = np.exp(qt[0] @ kk / np.sqrt(d))
        num = num + e * vv
        den = den + e
    np.testing.assert_allclose(out, num / den, rtol=1e-11)
    assert int(u.win_pos[-1]) == n and len(u.win_pos) == 4
    assert not np.array_equal(H, u.H)                      # the update ran before the output


# ------------------------------------------------------------------ I8: brute force on tiny inputs
def brute_force(q, k, v, W, eta, lam, C, kind, tail):
    """Independent restatement: where each past pair lives is kept in Python sets; the linear part
    is evaluated pair by pair through phi(a).phi(b) (never through a matrix H)."""
    g, n, d = q.shape
    scale = 1.0 / np.sqrt(d)
    fk = lib_phi(k, W, kind)
    in_win, in_G, in_H = [], set(), set()
    out = np.zeros((g, n, d))

    def lin_weights(fx):
        return {j: float(fx @ fk[j]) for j in in_H}

    def leave(R):
        nonlocal in_G, in_H
        cand = sorted(in_G) + list(R)
        if len(cand) <= lam:
            in_G = set(cand)
            return
        if lam == 0:
            in_H |= set(cand)
            in_G = set()
            return
        score = {}
        for c in cand:
            w = lin_weights(fk[c])
            tot = sum(w.values())
            vh = sum(w[j] * v[j] for j in in_H) / tot if tot > 0 else np.zeros(d)
            score[c] = float(np.linalg.norm(vh - v[c]))
        ranked = sorted(cand, key=lambda c: (-score[c], c))
        in_G = set(ranked[:lam])
        in_H |= set(ranked[lam:])

    def y(h, t, soft):
        fq = lib_phi(q[h, t:t + 1], W, kind)[0]
        w = lin_weights(fq)
        num = sum(w[j] * v[j] for j in in_H) if in_H else np.zeros(d)
        den = sum(w.values())
        for j in soft:
            e = np.exp(q[h, t] @ k[j] * scale)
            num = num + e * v[j]
            den += e
        return num / den

    t0 = 0
    while t0 < n - tail:
        c = min(C, n - tail - t0)
        for t in range(t0, t0 + c):
            soft = sorted(in_G) + in_win + list(range(t0, t + 1))
            for h in range(g):
                out[h, t] = y(h, t, soft)
        in_win = in_win + list(range(t0, t0 + c))
        over = max(0, len(in_win) - eta)
        R, in_win = in_win[:over], in_win[over:]
        leave(R)
        t0 += c
    for t in range(n - tail, n):
        in_win = in_win + [t]
        over = max(0, len(in_win) - eta)
        R, in_win = in_win[:over], in_win[over:]
        leave(R)
        for h in range(g):
            out[h, t] = y(h, t, sorted(in_G) + in_win)
    return out, in_win, in_G, in_H


@settings(max_examples=40, deadline=None)
@given(d=st.sampled_from([4, 8]), F=st.sampled_from([2, 4]), C=st.sampled_from([1, 2, 4]),
       eta_mult=st.sampled_from([0, 1, 2]), lam=st.sampled_from([0, 1, 3, 8]),
       n=st.integers(min_value=5, max_value=48), tail=st.integers(min_value=0, max_value=6),
       kind=st.sampled_from(["softmax", "exp"]), seed=st.integers(min_value=0, max_value=10 ** 6))
def test_brute_force_tiny(d, F, C, eta_mult, lam, n, tail, kind, seed):
    rng = np.random.default_rng(seed)
    eta = eta_mult * C
    tail = min(tail, n - 1)
    u, cfg, W = make_unit(d, F, eta=eta, lam=lam, kind=kind, rng=rng)
    q, k, v = rand_qkv(n, d, 2, rng=rng)
    if kind == "exp":
        q, k = 0.5 * q, 0.5 * k
    out = run_unit(u, q, k, v, C, decode_tail=tail)
    ref, win, G, Hset = brute_force(q, k, v, W, eta, lam, C, kind, tail)
    assert set(map(int, u.G_pos)) == G and set(u.folded_pos) == Hset and list(map(int, u.win_pos)) == win
    np.testing.assert_allclose(out, ref, rtol=1e-8, atol=1e-10)


# ------------------------------------------------------------------ I9: eager and lazy schedules agree
@pytest.mark.parametrize("eta,lam,C", [(8, 6, 8), (4, 3, 4), (6, 5, 3)])
def test_lazy_pseudocode_order_gives_same_outputs(eta, lam, C):
    d, F, n = 8, 4, 64
    rng = np.random.default_rng(3)
    W = rng.standard_normal((d, F)) / np.sqrt(d)
    q, k, v = rand_qkv(n, d, 2, rng=rng)
    a = UnitState(OracleConfig(1, 2, 1, d, F, eta, lam, schedule="eager"), W)
    b = UnitState(OracleConfig(1, 2, 1, d, F, eta, lam, schedule="lazy"), W)
    oa, ob = run_unit(a, q, k, v, C), run_unit(b, q, k, v, C)
    np.testing.assert_allclose(oa, ob, rtol=1e-12, atol=1e-14)
    # the lazy state is one eviction behind: it still holds the pairs the eager one just moved on
    assert len(b.win_pos) >= len(a.win_pos)
    assert set(map(int, a.folded_pos)) >= set(map(int, b.folded_pos))


# ------------------------------------------------------------------ W = 0: everything has a textbook value
def test_zero_feature_weights_running_mean():
    # phi is constant => the hidden state recalls the mean of the folded values for any key, and with
    # zero queries the output is the plain average over all past values (every weight equals 1).
    d, F, n, C, eta, lam = 8, 4, 30, 5, 5, 0
    cfg = OracleConfig(1, 1, 1, d, F, eta, lam)
    u = UnitState(cfg, np.zeros((d, F)))
    k, v = RNG.standard_normal((n, d)), RNG.standard_normal((n, d))
    q = np.zeros((1, n, d))
    out = run_unit(u, q, k, v, C)
    # weights: folded pair j contributes phi.phi = 2F * (1/F)^2 = 2/F ; softmax pairs contribute exp(0) = 1
    for t in [0, 7, 19, 29]:
        t0 = (t // C) * C
        w0 = max(0, t0 - eta)
        wts = np.array([2.0 / F] * w0 + [1.0] * (t + 1 - w0))
        np.testing.assert_allclose(out[0, t], (wts[:, None] * v[:t + 1]).sum(0) / wts.sum(), rtol=1e-12)


# ------------------------------------------------------------------ cache ablation (what the queries see)
@pytest.mark.parametrize("lin,sp", [(True, True), (False, True), (True, False), (False, False)])
def test_query_restrictions_change_eq14_only(lin, sp):
    """The ablation's flags leave the memories alone and drop exactly their terms from Eq. 14: outputs are
    recomputed from the raw arrays, the members' positions and H, s with unshifted exponentials; with both
    terms hidden the output is textbook softmax attention over the window and the causal part of the chunk."""
    d, F, eta, lam, C, n = 8, 4, 6, 5, 4, 48
    rng = np.random.default_rng(77)
    W = rng.standard_normal((d, F)) / np.sqrt(d)
    q, k, v = rand_qkv(n, d, 2, rng=rng)
    q, k, v = 0.5 * q, 0.5 * k, v
    full = UnitState(OracleConfig(1, 2, 1, d, F, eta, lam), W)
    abl = UnitState(OracleConfig(1, 2, 1, d, F, eta, lam, query_linear=lin, query_sparse=sp), W)
    scale = 1.0 / np.sqrt(d)
    for t0 in range(0, n, C):
        G_pos, H, s_ = abl.G_pos.copy(), abl.H.copy(), abl.s.copy()
        w0 = max(0, t0 - eta)
        out = abl.prefill_chunk(q[:, t0:t0 + C], k[t0:t0 + C], v[t0:t0 + C])
        full.prefill_chunk(q[:, t0:t0 + C], k[t0:t0 + C], v[t0:t0 + C])
        # the memories do not depend on what the queries see
        assert np.array_equal(abl.G_pos, full.G_pos) and np.array_equal(abl.H, full.H) and np.array_equal(abl.s, full.s)
        for hh in range(2):
            for r in range(C):
                t = t0 + r
                keys = list(range(w0, t + 1)) + (list(map(int, G_pos)) if sp else [])
                wts = np.exp(scale * (k[keys] @ q[hh, t]))
                num, den = wts @ v[keys], wts.sum()
                if lin:
                    fq = lib_phi(q[hh, t][None], W)[0]
                    num, den = num + fq @ H, den + fq @ s_
                np.testing.assert_allclose(out[hh, r], num / den, rtol=1e-10, atol=1e-12)
                if not lin and not sp:
                    keys = list(range(w0, t + 1))
                    ref = scipy.special.softmax(scale * (k[keys] @ q[hh, t])) @ v[keys]
                    np.testing.assert_allclose(out[hh, r], ref, rtol=1e-10, atol=1e-12)
    # generation steps: the new pair is in the window, the sparse cache is the updated one
    for t in range(n - 6, n):
        pass
    qd, kd, vd = rand_qkv(6, d, 2, rng=rng)
    for i in range(6):
        out = abl.decode_step(0.5 * qd[:, i], 0.5 * kd[i], vd[i])
        full.decode_step(0.5 * qd[:, i], 0.5 * kd[i], vd[i])
        assert np.array_equal(abl.G_pos, full.G_pos) and np.array_equal(abl.H, full.H)
        Ks = np.concatenate([abl.win_k] + ([abl.G_k] if sp else []), axis=0)
        Vs = np.concatenate([abl.win_v] + ([abl.G_v] if sp else []), axis=0)
        for hh in range(2):
            wts = np.exp(scale * (Ks @ (0.5 * qd[hh, i])))
            num, den = wts @ Vs, wts.sum()
            if lin:
                fq = lib_phi(0.5 * qd[hh, i][None], W)[0]
                num, den = num + fq @ abl.H, den + fq @ abl.s
            np.testing.assert_allclose(out[hh], num / den, rtol=1e-10, atol=1e-12)
