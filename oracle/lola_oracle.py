"""CPU oracle for the LoLA per-layer attention step (arXiv 2505.23666).

THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, float64 restatement of the
method written from the paper's equations, used only to check the CUDA library
and to be timed as the reported CPU baseline.  It shares no code with the CUDA
path and nothing in the product imports it.

What it follows (equation numbers count the paper's displayed equations in
order: (4) linear attention, (5) recurrent state update, (6) feature map,
(10) self-recall error, (11)-(13) eligible set / top-lambda / fold, (14) the
combined output with one shared denominator, (15) the chunkwise eligible set;
"pseudo-code" is the appendix "Algorithm Pseudo-Code"):

  phi            Eq. 6, and the softmax-halves variant the workloads use
  sre_scores     Eq. 10, against the state *before* the fold (pseudo-code order)
  evict          Eq. 11-13 and 15: score E = G u R, keep top-lambda, fold the rest
  attend_rows    Eq. 14
  prefill_chunk  section "Chunkwise Inference": attend, then evict
  decode_step    section "Mitigating Memory Collisions": update, then attend

Readings taken where the paper is silent:
  * exactly lambda pairs are kept; ties go to the older pair (lower position);
  * when |E| <= lambda nothing is scored or folded;  lambda = 0 folds everything;
  * if phi(k)^T s is not > 0 (only when s = 0) the predicted value is 0;
  * the exponentials of Eq. 14 are evaluated as exp(z - m) with m = max(0, max z)
    applied to all three terms, which leaves the quotient unchanged;
  * `operand_rounding="none"` (the default everywhere) is the method in float64
    on the inputs as given.  `operand_rounding="bf16"` is a diagnostic variant:
    phi(K_E) and H are rounded to bf16 as operands of the Eq. 10 contraction,
    which is what tensor-core operands of a bf16 library undergo; accumulation
    stays float64 and Eq. 13 folds phi(k) itself.  Tests use it beside the default
    to tell operand rounding apart from arithmetic mistakes.

Cache ablation (appendix "Sparse Cache & Linear Attention Ablation"): `query_linear=False` leaves the
phi(q)^T H and phi(q)^T s terms out of Eq. 14, `query_sparse=False` the sum over the sparse cache; the
memories are updated as always.

Parity pins: every function here is pinned by tests/test_oracle_pins.py
(closed forms, brute force, library special cases).  The absolute values of
outputs on the five full workloads have no external reference: for those,
parity is "GPU vs this oracle" only.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

try:  # keep BLAS single-threaded inside unit-level worker threads
    from threadpoolctl import threadpool_limits
except Exception:  # pragma: no cover
    threadpool_limits = None


# --------------------------------------------------------------------------- config
@dataclass
class OracleConfig:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    feat_half: int
    window: int                      # eta: pairs resident between calls
    sparse: int                      # lambda
    phi_kind: str = "softmax"        # "softmax" (workloads) | "exp" (Eq. 6)
    softmax_scale: Optional[float] = None   # None => 1/sqrt(head_dim) (Eq. 2)
    operand_rounding: str = "none"   # "none" | "bf16"
    schedule: str = "eager"          # "eager" | "lazy" (pseudo-code order of update_chunk)
    # cache ablation (appendix "Sparse Cache & Linear Attention Ablation"): what the QUERIES see in Eq. 14;
    # the memories are updated the same way whatever these say
    query_linear: bool = True        # the phi(q)^T H and phi(q)^T s terms
    query_sparse: bool = True        # the sum over the sparse cache G

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def feat_dim(self) -> int:
        return 2 * self.feat_half

    @property
    def scale(self) -> float:
        return (1.0 / np.sqrt(self.head_dim)) if self.softmax_scale is None else float(self.softmax_scale)


# --------------------------------------------------------------------------- arithmetic
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (8 significant bits, ties to even) of float64 data, as float64."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    u = x.view(np.uint64)
    drop = np.uint64(45)                                   # 52 - 7 mantissa bits
    r = (u + np.uint64((1 << 44) - 1) + ((u >> drop) & np.uint64(1))) & ~np.uint64((1 << 45) - 1)
    out = r.view(np.float64).reshape(x.shape).copy()
    tiny = np.abs(x) < 2.0 ** -126                         # bf16 subnormal range: fixed spacing 2^-133
    if np.any(tiny):
        out[tiny] = np.round(x[tiny] * 2.0 ** 133) * 2.0 ** -133
    return out


def phi(x: np.ndarray, W: np.ndarray, kind: str = "softmax") -> np.ndarray:
    """Feature map of rows x [n, d] with W [d, F] -> [n, 2F].

    "exp":     Eq. 6, [exp(xW), exp(-xW)].
    "softmax": each half normalised over its F entries, [softmax(xW), softmax(-xW)].
    """
    u = np.asarray(x, dtype=np.float64) @ np.asarray(W, dtype=np.float64)
    if kind == "exp":
        return np.concatenate([np.exp(u), np.exp(-u)], axis=-1)
    if kind != "softmax":
        raise ValueError(kind)
    a = np.exp(u - u.max(axis=-1, keepdims=True))
    b = np.exp(-u - (-u).max(axis=-1, keepdims=True))
    return np.concatenate([a / a.sum(-1, keepdims=True), b / b.sum(-1, keepdims=True)], axis=-1)


def sre_scores(f: np.ndarray, v: np.ndarray, H: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Self-recall error, Eq. 10: || f^T H / f^T s - v ||_2 per row (f = phi(k), [n, D])."""
    den = f @ s
    num = f @ H
    vhat = np.zeros_like(num)
    ok = den > 0
    vhat[ok] = num[ok] / den[ok, None]
    return np.sqrt(((vhat - v) ** 2).sum(axis=-1))


# --------------------------------------------------------------------------- one (batch row, KV head)
class UnitState:
    """The three memories of one attention head group (Fig. 1; pseudo-code `init`)."""

    def __init__(self, cfg: OracleConfig, W: np.ndarray):
        d, D = cfg.head_dim, cfg.feat_dim
        self.cfg = cfg
        self.W = np.asarray(W, dtype=np.float64)          # [d, F]
        self.win_pos = np.zeros((0,), dtype=np.int64)
        self.win_k = np.zeros((0, d))
        self.win_v = np.zeros((0, d))
        self.G_pos = np.zeros((0,), dtype=np.int64)
        self.G_k = np.zeros((0, d))
        self.G_v = np.zeros((0, d))
        self.G_score = np.zeros((0,))                      # SRE at the last update (nan: never scored)
        self.H = np.zeros((D, d))
        self.s = np.zeros((D,))
        self.n_seen = 0
        self.folded_pos: List[int] = []                    # bookkeeping for tests only
        self.last_kept_min = np.nan                        # lowest kept / highest folded score
        self.last_folded_max = np.nan                      # at the most recent scored update
        self.n_scored_updates = 0
        self.last_E_pos = np.zeros((0,), dtype=np.int64)   # eligible set and its scores at the most
        self.last_E_score = np.zeros((0,))                 # recent scored update (for tie-aware checks)

    # -- helpers
    def _rq(self, x: np.ndarray) -> np.ndarray:
        return round_bf16(x) if self.cfg.operand_rounding == "bf16" else x

    def _phi(self, x: np.ndarray) -> np.ndarray:
        return phi(x, self.W, self.cfg.phi_kind)

    # -- Eq. 11-13, 15
    def evict(self, R_pos: np.ndarray, R_k: np.ndarray, R_v: np.ndarray) -> None:
        """Pairs R leave the window (oldest first): E = G u R, keep top-lambda by SRE, fold the rest."""
        if len(R_pos) == 0:
            return
        lam = self.cfg.sparse
        E_pos = np.concatenate([self.G_pos, R_pos])
        E_k = np.concatenate([self.G_k, R_k], axis=0)
        E_v = np.concatenate([self.G_v, R_v], axis=0)
        m = len(E_pos)
        if m <= lam:                                        # below capacity: nothing scored, nothing folded
            self.G_pos, self.G_k, self.G_v = E_pos, E_k, E_v
            self.G_score = np.concatenate([self.G_score, np.full(len(R_pos), np.nan)])
            return
        f = self._phi(E_k)                                  # phi(K_E)
        if lam == 0:                                        # no sparse cache: everything folds, no scoring
            keep = np.zeros((0,), dtype=np.int64)
            lose = np.arange(m)
            score = np.full(m, np.nan)
        else:
            # state BEFORE this update's fold; the "bf16" variant rounds the two operands of this contraction only
            score = sre_scores(self._rq(f), E_v, self._rq(self.H), self.s)
            order = np.lexsort((E_pos, -score))             # score descending, then older first
            keep = np.sort(order[:lam])
            lose = np.sort(order[lam:])
            self.last_kept_min = float(score[keep].min())
            self.last_folded_max = float(score[lose].max())
            self.n_scored_updates += 1
            self.last_E_pos, self.last_E_score = E_pos.copy(), score.copy()
        # Eq. 13: H += sum phi(k) v^T, s += sum phi(k) over the pairs that are not kept
        self.H = self.H + f[lose].T @ E_v[lose]
        self.s = self.s + f[lose].sum(axis=0)
        self.folded_pos.extend(int(p) for p in E_pos[lose])
        self.G_pos, self.G_k, self.G_v, self.G_score = E_pos[keep], E_k[keep], E_v[keep], score[keep]

    # -- Eq. 14
    def attend_rows(self, q: np.ndarray, K: np.ndarray, V: np.ndarray, visible: np.ndarray) -> np.ndarray:
        """Eq. 14 for query rows q [r, d] over softmax keys K, V [n, d]; visible [r, n] bool.

        num = phi(q)^T H + sum_i exp(z_i) v_i,  den = phi(q)^T s + sum_i exp(z_i),  z = q.k / sqrt(d_k),
        each exponential written as exp(z - m) with the same factor exp(-m) on the linear terms.
        """
        fq = self._phi(q)                                   # [r, D]
        z = (q @ K.T) * self.cfg.scale if K.shape[0] else np.zeros((q.shape[0], 0))
        z = np.where(visible, z, -np.inf)
        m = np.maximum(0.0, z.max(axis=1, initial=-np.inf))
        w = np.exp(z - m[:, None])                          # masked entries: exp(-inf) = 0
        lin = np.exp(-m) if self.cfg.query_linear else np.zeros_like(m)
        num = lin[:, None] * (fq @ self.H) + w @ V
        den = lin * (fq @ self.s) + w.sum(axis=1)
        return num / den[:, None]

    def _pop_oldest(self, n_out: int):
        R = (self.win_pos[:n_out], self.win_k[:n_out], self.win_v[:n_out])
        self.win_pos, self.win_k, self.win_v = self.win_pos[n_out:], self.win_k[n_out:], self.win_v[n_out:]
        return R

    def _append(self, pos, k, v):
        self.win_pos = np.concatenate([self.win_pos, pos])
        self.win_k = np.concatenate([self.win_k, k], axis=0)
        self.win_v = np.concatenate([self.win_v, v], axis=0)

    # -- chunkwise inference: attend, then evict
    def prefill_chunk(self, q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
        """q [g, n, d], k, v [n, d] -> out [g, n, d].

        Every query of the chunk sees the resident window, the chunk causally (itself included),
        the sparse cache, and the H, s of the start of the call.  Afterwards the window takes the
        chunk and whatever exceeds eta leaves, oldest first, through `evict`.
        """
        cfg = self.cfg
        q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
        g, n, d = q.shape
        if cfg.schedule == "lazy":                          # pseudo-code order: evict first, then append
            over = max(0, len(self.win_pos) - cfg.window)
            self.evict(*self._pop_oldest(over))
        Gk, Gv = (self.G_k, self.G_v) if cfg.query_sparse else (self.G_k[:0], self.G_v[:0])
        K = np.concatenate([Gk, self.win_k, k], axis=0)
        V = np.concatenate([Gv, self.win_v, v], axis=0)
        n_old = len(Gk) + len(self.win_pos)
        vis = np.ones((n, n_old + n), dtype=bool)
        vis[:, n_old:] = np.tril(np.ones((n, n), dtype=bool))
        out = np.stack([self.attend_rows(q[h], K, V, vis) for h in range(g)], axis=0)
        self._append(np.arange(self.n_seen, self.n_seen + n, dtype=np.int64), k, v)
        self.n_seen += n
        if cfg.schedule == "eager":
            over = max(0, len(self.win_pos) - cfg.window)
            self.evict(*self._pop_oldest(over))
        return out

    # -- generation: update, then attend
    def decode_step(self, q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
        """q [g, d], k, v [d] -> out [g, d].  The new pair enters the window, the overflow is evicted
        (Eq. 11-13), then Eq. 14 runs over the updated caches, the new pair included."""
        cfg = self.cfg
        q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
        self._append(np.array([self.n_seen], dtype=np.int64), k[None, :], v[None, :])
        self.n_seen += 1
        over = max(0, len(self.win_pos) - cfg.window)
        self.evict(*self._pop_oldest(over))
        Gk, Gv = (self.G_k, self.G_v) if cfg.query_sparse else (self.G_k[:0], self.G_v[:0])
        K = np.concatenate([Gk, self.win_k], axis=0)
        V = np.concatenate([Gv, self.win_v], axis=0)
        vis = np.ones((q.shape[0], K.shape[0]), dtype=bool)
        return self.attend_rows(q, K, V, vis)


# --------------------------------------------------------------------------- batch of units
class LolaOracle:
    """All (batch row, KV head) units of one layer; units are independent."""

    def __init__(self, cfg: OracleConfig, W: np.ndarray, threads: int = 1):
        assert W.shape == (cfg.n_kv_heads, cfg.head_dim, cfg.feat_half), W.shape
        self.cfg = cfg
        self.units = [[UnitState(cfg, W[h]) for h in range(cfg.n_kv_heads)] for _ in range(cfg.batch)]
        self.threads = max(1, int(threads))
        self._pool = ThreadPoolExecutor(self.threads) if self.threads > 1 else None

    def _map(self, fn, items):
        if self._pool is None:
            return [fn(it) for it in items]
        if threadpool_limits is not None:
            with threadpool_limits(limits=1):
                return list(self._pool.map(fn, items))
        return list(self._pool.map(fn, items))

    def prefill_chunk(self, q, k, v, want_out: bool = True):
        """q [B, n, Hq, d], k, v [B, n, Hkv, d] -> out [B, n, Hq, d] float64 (None if not wanted:
        then only the caches advance, with a dummy query)."""
        cfg = self.cfg
        B, n = k.shape[0], k.shape[1]
        g = cfg.group
        out = np.zeros((B, n, cfg.n_q_heads, cfg.head_dim)) if want_out else None

        def work(bh):
            b, h = bh
            qq = (np.asarray(q[b, :, h * g:(h + 1) * g, :], dtype=np.float64).transpose(1, 0, 2)
                  if want_out else np.zeros((1, n, cfg.head_dim)))
            o = self.units[b][h].prefill_chunk(qq, k[b, :, h, :], v[b, :, h, :])
            if want_out:
                out[b, :, h * g:(h + 1) * g, :] = o.transpose(1, 0, 2)

        self._map(work, [(b, h) for b in range(B) for h in range(cfg.n_kv_heads)])
        return out

    def decode_step(self, q, k, v):
        """q [B, Hq, d], k, v [B, Hkv, d] -> out [B, Hq, d]."""
        cfg = self.cfg
        B = k.shape[0]
        g = cfg.group
        out = np.zeros((B, cfg.n_q_heads, cfg.head_dim))

        def work(bh):
            b, h = bh
            out[b, h * g:(h + 1) * g, :] = self.units[b][h].decode_step(q[b, h * g:(h + 1) * g, :], k[b, h], v[b, h])

        self._map(work, [(b, h) for b in range(B) for h in range(cfg.n_kv_heads)])
        return out

    def read_state(self) -> Dict[str, np.ndarray]:
        """Arrays in the layout of the library's state view (sparse slots in ascending position order)."""
        cfg = self.cfg
        B, Hk, d, D, lam, eta = cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.feat_dim, cfg.sparse, cfg.window
        wcap = max(1, max(len(u.win_pos) for row in self.units for u in row))
        st = {
            "H": np.zeros((B, Hk, D, d)), "s": np.zeros((B, Hk, D)),
            "sparse_count": np.zeros((B, Hk), dtype=np.int32),
            "sparse_pos": np.full((B, Hk, lam), -1, dtype=np.int64),
            "sparse_k": np.zeros((B, Hk, lam, d)), "sparse_v": np.zeros((B, Hk, lam, d)),
            "sparse_score": np.full((B, Hk, lam), np.nan),
            "window_count": np.zeros((B, Hk), dtype=np.int32),
            "window_pos": np.full((B, Hk, wcap), -1, dtype=np.int64),
            "window_k": np.zeros((B, Hk, wcap, d)), "window_v": np.zeros((B, Hk, wcap, d)),
            "threshold": np.full((B, Hk, 2), np.nan),
            "n_seen": np.zeros((B,), dtype=np.int64),
        }
        for b in range(B):
            for h in range(Hk):
                u = self.units[b][h]
                m, w = len(u.G_pos), len(u.win_pos)
                st["H"][b, h], st["s"][b, h] = u.H, u.s
                st["sparse_count"][b, h] = m
                st["sparse_pos"][b, h, :m] = u.G_pos
                st["sparse_k"][b, h, :m], st["sparse_v"][b, h, :m] = u.G_k, u.G_v
                st["sparse_score"][b, h, :m] = u.G_score
                st["window_count"][b, h] = w
                st["window_pos"][b, h, :w] = u.win_pos
                st["window_k"][b, h, :w], st["window_v"][b, h, :w] = u.win_k, u.win_v
                st["threshold"][b, h] = (u.last_kept_min, u.last_folded_max)
                st["n_seen"][b] = u.n_seen
        return st

    def needle_count(self, needle_pos: Sequence[int]) -> np.ndarray:
        """[B, Hkv] number of the given positions that sit in the sparse cache."""
        want = set(int(p) for p in needle_pos)
        return np.array([[sum(int(p) in want for p in u.G_pos) for u in row] for row in self.units], dtype=np.int64)


def config_for(wl, **kw) -> OracleConfig:
    """OracleConfig for a workload description (duck-typed: any object with the shape fields).
    The oracle is the method in float64 on the workload's (once-rounded) inputs; the operand roundings of
    the library's bf16 mode are an option the caller asks for (`operand_rounding="bf16"`)."""
    base = dict(batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                feat_half=wl.feat_half, window=wl.window, sparse=wl.sparse, operand_rounding="none")
    base.update(kw)
    return OracleConfig(**base)
