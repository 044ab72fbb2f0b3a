"""Lock-step comparison of the CUDA library with the CPU oracle on the same seeded inputs.

Both sides consume the same arrays call by call.  After every call the outputs are compared
element by element and the three memories are compared: sparse-cache membership must be identical
except where the oracle's own scores show a near-tie at the selection threshold; then the agreement
of the two sparse caches is recorded (Jaccard index per unit), the library's state is replaced by the
oracle's (oracle -> GPU, never the other way) and the run continues.  The number of such events is
reported and the callers bound it.

Two oracles serve the bf16 mode of the library:

  "plain"   float64 on the once-rounded inputs, no other rounding: the method itself.  The library's
            Eq. 10 contraction takes phi(K) and H rounded to bf16, so its scores differ from this
            oracle's by the rounding of those operands, and pairs whose score lies within that
            distance of the threshold may land on either side.
  "mirror"  the same oracle with phi(K_E) and H rounded to bf16 as operands of Eq. 10 (the roundings the
            library's tensor-core operands undergo there; accumulation stays float64; Eq. 13 folds phi(k)
            itself in both).  A diagnostic of the kernels' arithmetic: scores then agree to fp32
            accumulation error, so the near-tie band is an order of magnitude tighter.

Tolerances:
  fp32 mode:        |gpu - ref| <= 1e-4 * (|ref| + mean|ref|) for outputs, H and s; membership exact except
                    pairs whose oracle score lies within 1e-5 * max(1, |tau|) of the threshold tau.
  bf16 vs plain:    |gpu - ref| <= 2e-2 for outputs and H (s: 2e-2 relative to its scale); member scores
                    and near-ties within 3e-4 * max(1, |tau|).  One unit in the last place of a bf16
                    operand moves a term of phi(k)^T H by 2^-9 of its size; the 128 terms of a column add up
                    with independent signs, so the error norm moves by about 2^-9 * |v| / sqrt(128) ~ 2e-4 |tau|
                    at |tau| ~ |v|.  Measured on the five workloads: member scores within 1.2e-4 * |tau|,
                    swapped pairs within 1.4e-5 * |tau| of the threshold.
  bf16 vs mirror:   outputs and H as above; member scores and near-ties within 1e-4 * max(1, |tau|)
                    (measured: 1.3e-5 in the prefill kernels, 3.7e-5 in the fused generation step, whose
                    normaliser and error norm are summed in another order; swapped pairs within 2e-7).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle.lola_oracle import LolaOracle, config_for
from paper_2505_23666_b200 import binding
from paper_2505_23666_b200.workloads import Workload, WorkloadInputs

BF16_MODES = ("plain", "mirror")


def tolerances(dtype: str, oracle_mode: str = "plain"):
    if dtype == "bf16":
        band = 3e-4 if oracle_mode == "plain" else 1e-4
        return dict(kind="abs", out=2e-2, H=2e-2, tie=band, score=band)
    return dict(kind="rel", out=1e-4, H=1e-4, tie=1e-5, score=1e-4)


def close(gpu: np.ndarray, ref: np.ndarray, tol: float, kind: str):
    """Returns (ok, worst ratio of error to allowance)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(gpu - ref)
    if kind == "rel":
        allow = tol * (np.abs(ref) + np.abs(ref).mean() + 1e-30)
    else:
        allow = np.full_like(err, tol)
    ratio = float((err / allow).max()) if err.size else 0.0
    return bool(np.isfinite(gpu).all() and ratio <= 1.0), ratio


def oracle_for(wl: Workload, inputs: WorkloadInputs, batch: int, oracle_mode: str = "plain", threads: int = 8, **kw):
    rounding = "bf16" if (wl.dtype == "bf16" and oracle_mode == "mirror") else "none"
    ocfg = config_for(wl, batch=batch, operand_rounding=rounding, **kw)
    return LolaOracle(ocfg, inputs.W.astype(np.float64), threads=threads)


def compare_unit(g, u, b, h, tol, where, worst):
    """One unit of a library state view `g` against the oracle's unit state `u`.
    Returns None when everything agrees, else the library's member set when only the membership
    differs; asserts on anything else."""
    m, w = len(u.G_pos), len(u.win_pos)
    assert int(g["sparse_count"][b, h]) == m, f"{where}: sparse counts differ"
    assert int(g["window_count"][b, h]) == w, f"{where}: window counts differ"
    gp = g["window_pos"][b, h]
    sel = gp >= 0
    order = np.argsort(gp[sel])
    assert np.array_equal(gp[sel][order], u.win_pos), f"{where}: window positions"
    assert np.array_equal(g["window_k"][b, h][sel][order], u.win_k.astype(np.float32)), where
    assert np.array_equal(g["window_v"][b, h][sel][order], u.win_v.astype(np.float32)), where
    gpos = g["sparse_pos"][b, h, :m].astype(np.int64)
    assert np.all(g["sparse_pos"][b, h, m:] == -1), f"{where}: stale slots"
    assert len(set(gpos.tolist())) == m, f"{where}: duplicate members"
    so = np.argsort(gpos)
    if not np.array_equal(gpos[so], u.G_pos):               # (the oracle keeps its members in ascending position order)
        return set(gpos.tolist())
    assert np.array_equal(g["sparse_k"][b, h, :m][so], u.G_k.astype(np.float32)), where
    assert np.array_equal(g["sparse_v"][b, h, :m][so], u.G_v.astype(np.float32)), where
    for name, ref in (("H", u.H), ("s", u.s)):
        t = tol["H"]
        if name == "s" and tol["kind"] == "abs":
            t = tol["H"] * max(1.0, float(np.abs(ref).max()))
        ok, ratio = close(g[name][b, h], ref, t, tol["kind"])
        worst[name] = max(worst[name], ratio)
        assert ok, f"{where}: {name} of unit ({b},{h}) outside tolerance ({ratio:.3g})"
    # scores of the members, where both sides have scored them
    gs, os_ = g["sparse_score"][b, h, :m][so], u.G_score
    both = ~np.isnan(os_)
    assert np.array_equal(np.isnan(gs), np.isnan(os_)), f"{where}: scored/unscored flags"
    if both.any():
        ratio = float((np.abs(gs[both] - os_[both]) / (tol["score"] * np.maximum(1.0, np.abs(os_[both])))).max())
        worst["score"] = max(worst["score"], ratio)
        assert ratio <= 1.0, f"{where}: member scores differ ({ratio:.3g} of the allowance)"
    return None


def assert_near_tie(u, gpu_members: set, tie: float, where, unit, worst=None):
    """Membership differs: every pair on the wrong side must be a near-tie in the ORACLE's scores of
    this update, and the difference must be a swap of equal numbers of pairs.  Returns the Jaccard
    index of the two member sets."""
    orc_members = set(int(p) for p in u.G_pos)
    only_g, only_o = gpu_members - orc_members, orc_members - gpu_members
    assert len(only_g) == len(only_o) > 0, f"{where} unit {unit}: membership sizes differ"
    sc = {int(p): float(s) for p, s in zip(u.last_E_pos, u.last_E_score)}
    tau = 0.5 * (u.last_kept_min + u.last_folded_max)
    band = tie * max(1.0, abs(tau))
    for p in sorted(only_g | only_o):
        assert p in sc, f"{where} unit {unit}: pair {p} was not eligible in this update"
        if worst is not None:
            worst["tie"] = max(worst.get("tie", 0.0), abs(sc[p] - tau) / band)
        assert abs(sc[p] - tau) <= band, \
            f"{where} unit {unit}: pair {p} differs and is no near-tie (score {sc[p]:.9g}, threshold {tau:.9g})"
    return len(gpu_members & orc_members) / max(1, len(gpu_members | orc_members))


class Lockstep:
    def __init__(self, wl: Workload, rows=None, threads: int = 8, device="cuda:0", inputs: WorkloadInputs = None,
                 generic_kernels: bool = False, softmax_scale: float = 0.0, oracle_mode: str = "plain",
                 phi_kind: str = "softmax", flags: int = 0):
        self.wl = wl
        self.rows = list(range(wl.batch)) if rows is None else list(rows)
        self.inputs = inputs or WorkloadInputs(wl)
        B = len(self.rows)
        self.oracle_mode = oracle_mode
        self.tol = tolerances(wl.dtype, oracle_mode)
        self.oracle = oracle_for(wl, self.inputs, B, oracle_mode, threads, softmax_scale=(softmax_scale or None),
                                 phi_kind=phi_kind, query_linear=not (flags & binding.LOLA_FLAG_QUERY_NO_LINEAR),
                                 query_sparse=not (flags & binding.LOLA_FLAG_QUERY_NO_SPARSE))
        self.ocfg = self.oracle.cfg
        self.cfg = binding.make_config(B, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.feat_half, wl.window,
                                       wl.sparse, max(wl.chunk, 1), dtype=wl.dtype, generic_kernels=generic_kernels,
                                       softmax_scale=softmax_scale, phi_kind=phi_kind, flags=flags)
        self.layer = binding.LolaLayer(self.cfg, self.inputs.W, device=device)
        self.resyncs = 0
        self.diverged_units = 0
        self.min_jaccard = 1.0
        self.scored_updates = 0
        self.worst = {"out": 0.0, "H": 0.0, "s": 0.0, "score": 0.0, "tie": 0.0}
        self.calls = 0

    # ------------------------------------------------------------------ steps
    def prefill(self, t0: int, n: int, want_out: bool = True, check_state=True):
        """check_state: True = all memories, "members" = sparse-cache membership only (full check of a unit
        whose membership differs), False = nothing."""
        q, k, v = self.inputs.prefill_tokens(t0, n, batch_rows=self.rows, need_q=want_out)
        L = self.layer
        dq = L.to_device(q) if want_out else None
        out = L.prefill_chunk(dq, L.to_device(k), L.to_device(v), want_out=want_out)
        ref = self.oracle.prefill_chunk(q, k, v, want_out=want_out)
        if want_out:
            self._cmp_out(out.float().cpu().numpy(), ref, f"prefill t0={t0}")
        self.calls += 1
        if check_state:
            self.check_state(f"prefill t0={t0}", members_only=(check_state == "members"))

    def decode(self, step: int, check_state: bool = True):
        q, k, v = self.inputs.decode_token(step, batch_rows=self.rows)
        L = self.layer
        out = L.decode_step(L.to_device(q), L.to_device(k), L.to_device(v)).float().cpu().numpy()
        ref = self.oracle.decode_step(q, k, v)
        self.calls += 1
        # A generation step selects first and attends afterwards, so where the two sides resolved a
        # near-tie differently (verified against the oracle's own scores in check_state) their outputs
        # of this step answer different, equally valid, cache contents: those units are not compared.
        diverged = self.check_state(f"decode step={step}") if check_state else []
        g = self.wl.group
        for (b, h) in diverged:
            out[b, h * g:(h + 1) * g] = ref[b, h * g:(h + 1) * g]
        self._cmp_out(out, ref, f"decode step={step}")

    # ------------------------------------------------------------------ comparisons
    def _cmp_out(self, gpu, ref, where):
        ok, ratio = close(gpu, ref, self.tol["out"], self.tol["kind"])
        self.worst["out"] = max(self.worst["out"], ratio)
        assert ok, f"{where}: output outside tolerance (worst error/allowance {ratio:.3g})"

    def check_state(self, where: str = "", members_only: bool = False):
        units = self.oracle.units
        B, Hk = len(units), len(units[0])
        self.scored_updates = sum(u.n_scored_updates for row in units for u in row)
        if members_only:
            g = self.layer.read_state(fields=("sparse_pos", "status"))
            assert int(g["status"][0]) == 0, f"{where}: device status {int(g['status'][0])}"
            if all(np.array_equal(np.sort(g["sparse_pos"][b, h, :len(units[b][h].G_pos)].astype(np.int64)), units[b][h].G_pos)
                   for b in range(B) for h in range(Hk)):
                return []
        g = self.layer.read_state()
        assert int(g["status"][0]) == 0, f"{where}: device status {int(g['status'][0])}"
        assert all(int(n) == units[0][0].n_seen for n in g["n_seen"]), where
        diverged = []
        for b in range(B):
            for h in range(Hk):
                u = units[b][h]
                members = compare_unit(g, u, b, h, self.tol, where, self.worst)
                if members is not None:
                    jac = assert_near_tie(u, members, self.tol["tie"], where, (b, h), self.worst)
                    self.min_jaccard = min(self.min_jaccard, jac)
                    diverged.append((b, h))
        if diverged:
            self.resyncs += 1
            self.diverged_units += len(diverged)
            self.layer.write_state(self.oracle.read_state())
        return diverged

    def summary(self):
        return dict(oracle=self.oracle_mode, calls=self.calls, resyncs=self.resyncs, diverged_units=self.diverged_units,
                    min_jaccard=self.min_jaccard, scored_updates=self.scored_updates, worst=dict(self.worst))
