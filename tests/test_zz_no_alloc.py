"""lola_decode_step_static: the generation step for callers that cannot hand the library scratch memory
(device allocation closed after start-up).  Its work lists sit in a static device array inside the
library instead of the caller's state buffer; everything else is the same step, so its outputs and
the state it leaves must equal those of lola_decode_step.  Checked on two calls in a row (the array
is shared and keeps the previous call's contents), through the C ABI, and for the size limit.
This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2505_23666_b200 import binding as b
from paper_2505_23666_b200.workloads import WorkloadInputs, small_case

pytestmark = pytest.mark.gpu


def _prefilled(wl, inp):
    cfg = b.make_config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.feat_half, wl.window, wl.sparse,
                        wl.chunk, dtype=wl.dtype)
    layer = b.LolaLayer(cfg, inp.W)
    for t in range(0, wl.tokens, wl.chunk):
        _, k, v = inp.prefill_tokens(t, wl.chunk, need_q=False)
        layer.prefill_chunk(None, layer.to_device(k), layer.to_device(v), want_out=False)
    return layer


def test_static_scratch_decode_matches_fused_decode():
    """At shapes where lola_decode_step runs as the single fused kernel (bf16, lambda a multiple of 64) the
    static variant runs the kernel chain instead: same step, other kernels, so outputs agree to the bf16
    tolerance, not bit for bit.  A unit where the two resolved a tie at the selection threshold differently
    (the reference's lowest kept and highest folded scores within 1e-4 of each other) is left out."""
    wl = small_case("noalloc128", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, feat_half=64, tokens=384, chunk=64,
                    window=64, sparse=128, dtype="bf16", seed=22)
    inp = WorkloadInputs(wl)
    ref, new = _prefilled(wl, inp), _prefilled(wl, inp)
    s = torch.cuda.current_stream().cuda_stream
    g = wl.group
    for step in range(4):
        q, k, v = (ref.to_device(a) for a in inp.decode_token(step))
        out_ref, out_new = torch.empty_like(q), torch.full_like(q, float("nan"))
        assert b.lola_decode_step(ref.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out_ref.data_ptr(), s) == b.LOLA_OK
        assert "decode_fused" in ref.last_call_info()["paths"]
        assert b.lola_decode_step_static(new.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out_new.data_ptr(), s) == b.LOLA_OK
        assert "decode_fused" not in new.last_call_info()["paths"]
        torch.cuda.synchronize()
        a, c = ref.read_state(), new.read_state()
        assert int(c["status"][0]) == 0
        resync = False
        for bi in range(wl.batch):
            for h in range(wl.n_kv_heads):
                if set(a["sparse_pos"][bi, h].tolist()) != set(c["sparse_pos"][bi, h].tolist()):
                    kept, folded = a["threshold"][bi, h]
                    assert abs(kept - folded) <= 1e-4 * max(1.0, abs(kept)), (step, bi, h, kept, folded)
                    resync = True
                    continue
                err = (out_new[bi, h * g:(h + 1) * g].float() - out_ref[bi, h * g:(h + 1) * g].float()).abs().max().item()
                assert err <= 2e-2, (step, bi, h, err)
                assert np.abs(c["H"][bi, h] - a["H"][bi, h]).max() <= 2e-2
        for key in ("window_k", "window_v", "n_seen"):
            assert np.array_equal(a[key], c[key]), key
        if resync:
            new.write_state(a)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_scratch_decode_matches_decode(dtype):
    wl = small_case("noalloc", batch=3, n_q_heads=4, n_kv_heads=2, head_dim=64, feat_half=64, tokens=256, chunk=32,
                    window=32, sparse=40, dtype=dtype, seed=21, scale_a=(0.125 if dtype == "f32" else 1.0))
    inp = WorkloadInputs(wl)
    ref, new = _prefilled(wl, inp), _prefilled(wl, inp)
    s = torch.cuda.current_stream().cuda_stream
    for step in range(2):                                   # two calls in a row share the static array
        q, k, v = (ref.to_device(a) for a in inp.decode_token(step))
        out_ref, out_new = torch.empty_like(q), torch.full_like(q, float("nan"))
        assert b.lola_decode_step(ref.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out_ref.data_ptr(), s) == b.LOLA_OK
        assert b.lola_decode_step_static(new.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out_new.data_ptr(), s) == b.LOLA_OK
        torch.cuda.synchronize()
        tol = 2e-2 if dtype == "bf16" else 1e-4 * (out_ref.float().abs().mean().item() + 1e-30)
        assert torch.isfinite(out_new.float()).all()
        assert (out_new.float() - out_ref.float()).abs().max().item() <= tol
        a, c = ref.read_state(), new.read_state()
        for key in ("sparse_pos", "sparse_k", "sparse_v", "window_k", "window_v", "n_seen"):
            assert np.array_equal(a[key], c[key]), key
        np.testing.assert_allclose(c["H"], a["H"], rtol=1e-4, atol=(2e-2 if dtype == "bf16" else 1e-7))
        np.testing.assert_allclose(c["s"], a["s"], rtol=1e-4, atol=1e-6)
        assert int(c["status"][0]) == 0


def test_static_scratch_decode_rejects_oversize_states():
    # 8 x 2 units x max_chunk 8192 = 131072 list entries > LOLA_STATIC_MAX_LIST_ENTRIES (65536)
    cfg = b.make_config(8, 2, 2, 64, 64, 4, 4, 8192, dtype="f32")
    layer = b.LolaLayer(cfg, np.zeros((2, 64, 64), np.float32))
    x = torch.zeros((8, 2, 64), device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    rc = b.lola_decode_step_static(layer.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), s)
    assert rc == b.LOLA_ERR_SIZE and layer.tokens_seen == 0
    assert b.lola_decode_step_static(None, 0, 0, 0, 0, None) == b.LOLA_ERR_ARG
