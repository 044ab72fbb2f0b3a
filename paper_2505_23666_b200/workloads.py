"""Seeded synthetic inputs for the five LoLA workloads.

This module only draws random numbers and shapes them.  It holds none of the
method's arithmetic (no feature map, no attention, no scoring): both the CPU
oracle's tests and the CUDA path's tests/benchmarks read their inputs from
here, and nothing else is shared between the two.

Streams are keyed with Philox counters by (seed, batch row, cell index) so a
long sequence can be produced cell by cell (a cell is `cell_tokens` consecutive
tokens of one batch row) and so that one batch row can be generated without
generating the others (the units of the method are independent, which is what
lets a test check a sampled subset of a full-size run).

Recipe (the paper measures on trained-model activations of Llama-3.2-1B /
Llama-3.1-8B shape and on pass-key retrieval prompts; these inputs stand in for
their shapes only):
  * W[h] in R^{d x F}, iid N(0, 1/d), one per KV head.
  * 16 cluster centres mu[h][c] in R^d, iid N(0, I), per KV head.
  * key  = (mu[cluster] + 0.3 * eps) * a, cluster uniform in 0..15, eps ~ N(0, I)
  * query, value = N(0, I) * a;  a = 1/sqrt(64) for workload 0, 1 otherwise.
  * workload 4: 32 "needle" positions, uniform without replacement in
    [0, tokens-128); there each KV head's key is a random vector made
    orthogonal to that head's 16 centres and scaled to unit norm, the value is
    N(0, I); the last 32 queries of the sequence are copies of the needle keys.
  * bf16 workloads round every array once, here, to the nearest bf16 value
    (ties to even) and hand it out as float32 holding exactly that value.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

N_CLUSTERS = 16
CLUSTER_SIGMA = 0.3
N_NEEDLES = 32

# Philox stream ids (third counter word)
_STREAM_STATIC, _STREAM_KV, _STREAM_Q, _STREAM_NEEDLE, _STREAM_DECODE = 1, 2, 3, 4, 5


@dataclass(frozen=True)
class Workload:
    """Shape, cache sizes and input recipe of one workload."""
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    feat_half: int          # F; the feature map has D = 2F outputs
    tokens: int             # prefill length
    chunk: int              # C
    window: int             # eta
    sparse: int             # lambda
    dtype: str              # "f32" | "bf16"
    seed: int
    scale_a: float = 1.0
    decode_steps: int = 0   # single-token steps after the prefill
    needles: int = 0
    cell_tokens: int = 64   # generation granularity (independent of `chunk`)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def feat_dim(self) -> int:
        return 2 * self.feat_half

    @property
    def units(self) -> int:
        return self.batch * self.n_kv_heads

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # tiny single layer, fp32
    "cfg0": Workload("cfg0", 1, 4, 4, 64, 64, 1024, 64, 64, 128, "f32", 0, scale_a=1.0 / 8.0),
    # Llama-3.2-1B-shaped layer
    "cfg1": Workload("cfg1", 1, 32, 8, 64, 64, 4096, 64, 64, 512, "bf16", 1),
    # Llama-3.1-8B-shaped layer, batch 8
    "cfg2": Workload("cfg2", 8, 32, 8, 128, 64, 4096, 64, 64, 832, "bf16", 2),
    # decode batch, 8B shapes
    "cfg3": Workload("cfg3", 64, 32, 8, 128, 64, 32768, 64, 64, 832, "bf16", 3, decode_steps=256),
    # long-context pass-key-shaped
    "cfg4": Workload("cfg4", 1, 32, 8, 128, 64, 131072, 64, 64, 832, "bf16", 4, needles=N_NEEDLES),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float32 values to bf16, returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def _rng(seed: int, stream: int, a: int = 0, b: int = 0) -> np.random.Generator:
    # key = (seed, salt); counter = (0, stream, a, b): distinct (stream, a, b)
    # start 2^64 blocks apart, so streams never overlap.
    bitgen = np.random.Philox(key=[seed, 0x10A_2505_23666], counter=[0, stream, a, b])
    return np.random.Generator(bitgen)


class WorkloadInputs:
    """Seeded generator of one workload's arrays.

    Static arrays: `W` [Hkv, d, F], `centres` [Hkv, 16, d], `needle_pos` [needles]
    (sorted), `needle_k` [needles, Hkv, d], `needle_v` [needles, Hkv, d].
    All returned arrays are float32 (already rounded to bf16 values when the
    workload's dtype is bf16).
    """

    def __init__(self, wl: Workload):
        self.wl = wl
        d, F, Hkv = wl.head_dim, wl.feat_half, wl.n_kv_heads
        g = _rng(wl.seed, _STREAM_STATIC)
        W = g.standard_normal((Hkv, d, F), dtype=np.float32) * np.float32(1.0 / np.sqrt(d))
        self.centres = g.standard_normal((Hkv, N_CLUSTERS, d), dtype=np.float32)
        self.W = self._q(W)
        self.needle_pos = np.zeros((0,), dtype=np.int64)
        self.needle_k = np.zeros((0, Hkv, d), dtype=np.float32)
        self.needle_v = np.zeros((0, Hkv, d), dtype=np.float32)
        if wl.needles:
            gn = _rng(wl.seed, _STREAM_NEEDLE)
            hi = wl.tokens - 128
            self.needle_pos = np.sort(gn.choice(hi, size=wl.needles, replace=False)).astype(np.int64)
            raw = gn.standard_normal((wl.needles, Hkv, d)).astype(np.float64)
            nk = np.empty_like(raw)
            for h in range(Hkv):
                # orthonormal basis of the span of this head's centres
                qb, _ = np.linalg.qr(self.centres[h].astype(np.float64).T)   # [d, 16]
                r = raw[:, h, :] - (raw[:, h, :] @ qb) @ qb.T
                nk[:, h, :] = r / np.linalg.norm(r, axis=1, keepdims=True)
            self.needle_k = self._q(nk.astype(np.float32))
            self.needle_v = self._q(gn.standard_normal((wl.needles, Hkv, d), dtype=np.float32))

    # -- helpers -----------------------------------------------------------
    def _q(self, x: np.ndarray) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.float32)
        return round_to_bf16(x) if self.wl.dtype == "bf16" else x

    def _cell_kv(self, b: int, cell: int) -> Tuple[np.ndarray, np.ndarray]:
        wl = self.wl
        T, Hkv, d = wl.cell_tokens, wl.n_kv_heads, wl.head_dim
        g = _rng(wl.seed, _STREAM_KV, cell, b)
        cl = g.integers(0, N_CLUSTERS, size=(T, Hkv))
        eps = g.standard_normal((T, Hkv, d), dtype=np.float32)
        v = g.standard_normal((T, Hkv, d), dtype=np.float32)
        mu = self.centres[np.arange(Hkv)[None, :], cl]              # [T, Hkv, d]
        a = np.float32(wl.scale_a)
        k = (mu + np.float32(CLUSTER_SIGMA) * eps) * a
        v = v * a
        if wl.needles:
            t0 = cell * T
            for i, p in enumerate(self.needle_pos):
                if t0 <= p < t0 + T:
                    k[p - t0] = self.needle_k[i]
                    v[p - t0] = self.needle_v[i]
        return self._q(k), self._q(v)

    def _cell_q(self, b: int, cell: int) -> np.ndarray:
        wl = self.wl
        T = wl.cell_tokens
        g = _rng(wl.seed, _STREAM_Q, cell, b)
        q = g.standard_normal((T, wl.n_q_heads, wl.head_dim), dtype=np.float32) * np.float32(wl.scale_a)
        if wl.needles:
            # the last `needles` queries of the sequence look the needles up
            t0 = cell * T
            first = wl.tokens - wl.needles
            for i in range(wl.needles):
                p = first + i
                if t0 <= p < t0 + T:
                    q[p - t0] = np.repeat(self.needle_k[i], wl.group, axis=0)
        return self._q(q)

    # -- public ------------------------------------------------------------
    def prefill_tokens(self, t0: int, n: int, batch_rows: Optional[List[int]] = None,
                       need_q: bool = True):
        """Tokens [t0, t0+n) of the prefill for the given batch rows (default all).

        Returns (q, k, v): q [B', n, Hq, d] (or None), k and v [B', n, Hkv, d].
        """
        wl = self.wl
        rows = list(range(wl.batch)) if batch_rows is None else list(batch_rows)
        assert 0 <= t0 and t0 + n <= wl.tokens
        T = wl.cell_tokens
        c0, c1 = t0 // T, (t0 + n - 1) // T
        qs, ks, vs = [], [], []
        for b in rows:
            kk, vv, qq = [], [], []
            for c in range(c0, c1 + 1):
                k, v = self._cell_kv(b, c)
                kk.append(k)
                vv.append(v)
                if need_q:
                    qq.append(self._cell_q(b, c))
            lo = t0 - c0 * T
            ks.append(np.concatenate(kk, 0)[lo:lo + n])
            vs.append(np.concatenate(vv, 0)[lo:lo + n])
            if need_q:
                qs.append(np.concatenate(qq, 0)[lo:lo + n])
        q = np.ascontiguousarray(np.stack(qs, 0)) if need_q else None
        return q, np.ascontiguousarray(np.stack(ks, 0)), np.ascontiguousarray(np.stack(vs, 0))

    def decode_token(self, step: int, batch_rows: Optional[List[int]] = None):
        """Inputs of single-token step `step` after the prefill.

        Returns (q [B', Hq, d], k [B', Hkv, d], v [B', Hkv, d]).
        """
        wl = self.wl
        rows = list(range(wl.batch)) if batch_rows is None else list(batch_rows)
        Hq, Hkv, d = wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        a = np.float32(wl.scale_a)
        qs, ks, vs = [], [], []
        for b in rows:
            g = _rng(wl.seed, _STREAM_DECODE, step, b)
            cl = g.integers(0, N_CLUSTERS, size=(Hkv,))
            eps = g.standard_normal((Hkv, d), dtype=np.float32)
            v = g.standard_normal((Hkv, d), dtype=np.float32) * a
            q = g.standard_normal((Hq, d), dtype=np.float32) * a
            k = (self.centres[np.arange(Hkv), cl] + np.float32(CLUSTER_SIGMA) * eps) * a
            qs.append(q)
            ks.append(k)
            vs.append(v)
        return self._q(np.stack(qs, 0)), self._q(np.stack(ks, 0)), self._q(np.stack(vs, 0))


def small_case(name: str = "small", *, batch=2, n_q_heads=4, n_kv_heads=2, head_dim=64, feat_half=64,
               tokens=256, chunk=32, window=32, sparse=48, dtype="f32", seed=7, scale_a=1.0,
               decode_steps=0, needles=0, cell_tokens=64) -> Workload:
    """A reduced workload with the same recipe, for tests."""
    return Workload(name, batch, n_q_heads, n_kv_heads, head_dim, feat_half, tokens, chunk, window,
                    sparse, dtype, seed, scale_a=scale_a, decode_steps=decode_steps, needles=needles,
                    cell_tokens=cell_tokens)
