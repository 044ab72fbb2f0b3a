"""The seeded input generator: determinism, independence of batch rows and cells, recipe shapes."""
import numpy as np
import pytest

from paper_2505_23666_b200.workloads import (WORKLOADS, WorkloadInputs, round_to_bf16, small_case)


def test_cells_and_rows_are_independent_and_repeatable():
    wl = small_case(batch=3, tokens=512, dtype="bf16")
    a, b = WorkloadInputs(wl), WorkloadInputs(wl)
    q1, k1, v1 = a.prefill_tokens(0, 512)
    q2, k2, v2 = b.prefill_tokens(100, 200, batch_rows=[2])
    np.testing.assert_array_equal(q1[2:3, 100:300], q2)
    np.testing.assert_array_equal(k1[2:3, 100:300], k2)
    np.testing.assert_array_equal(v1[2:3, 100:300], v2)
    _, k3, v3 = a.prefill_tokens(100, 200, batch_rows=[2], need_q=False)
    np.testing.assert_array_equal(k3, k2)
    assert not np.array_equal(k1[0], k1[1])
    # bf16 workloads hold exactly representable values
    np.testing.assert_array_equal(round_to_bf16(k1), k1)
    np.testing.assert_array_equal(round_to_bf16(a.W), a.W)


def test_round_to_bf16_matches_torch():
    import torch
    x = (np.random.default_rng(0).standard_normal(4096) * 37).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(round_to_bf16(x), ref)


def test_recipe_statistics():
    wl = WORKLOADS["cfg1"]
    g = WorkloadInputs(wl)
    assert g.W.shape == (8, 64, 64) and abs(g.W.std() - 1 / 8) < 5e-3
    q, k, v = g.prefill_tokens(0, 512)
    assert q.shape == (1, 512, 32, 64) and k.shape == (1, 512, 8, 64)
    assert abs(q.std() - 1) < 0.02 and abs(v.std() - 1) < 0.02
    # keys sit near one of the 16 centres of their head
    dist = np.linalg.norm(k[0, :, 3, None, :] - g.centres[3][None], axis=-1).min(axis=1)
    assert np.all(dist < 0.3 * np.sqrt(64) * 1.6)
    w0 = WorkloadInputs(WORKLOADS["cfg0"])
    q0, k0, v0 = w0.prefill_tokens(0, 256)
    assert abs(q0.std() - 1 / 8) < 5e-3 and q0.dtype == np.float32


def test_needles_are_planted_and_queried():
    wl = small_case(batch=1, n_q_heads=4, n_kv_heads=2, tokens=512, needles=32, dtype="bf16")
    g = WorkloadInputs(wl)
    assert len(set(g.needle_pos.tolist())) == 32 and g.needle_pos.max() < 512 - 128
    q, k, v = g.prefill_tokens(0, 512)
    for i, p in enumerate(g.needle_pos):
        np.testing.assert_array_equal(k[0, p], g.needle_k[i])
        np.testing.assert_array_equal(v[0, p], g.needle_v[i])
        np.testing.assert_array_equal(q[0, 512 - 32 + i, 2], g.needle_k[i, 1])
    nk = g.needle_k.astype(np.float64)
    assert np.allclose(np.linalg.norm(nk, axis=-1), 1.0, atol=1e-2)
    for h in range(2):
        assert np.abs(nk[:, h] @ g.centres[h].astype(np.float64).T).max() < 5e-2


def test_decode_tokens():
    g = WorkloadInputs(small_case(batch=2, decode_steps=4))
    q, k, v = g.decode_token(3)
    q2, k2, v2 = g.decode_token(3, batch_rows=[1])
    assert q.shape == (2, 4, 64) and k.shape == (2, 2, 64)
    np.testing.assert_array_equal(q[1:], q2)
    np.testing.assert_array_equal(k[1:], k2)
