"""The context-free decode entry point (no allocation inside the library) against the regular one.

Some callers cannot allocate device memory at all - a plug-in in a process whose pool already owns the
device, or code running next to an open stream capture - so they cannot create a library context.  For them
bpc_decode_attn_static keeps its index list and error word in an array built into the library.  This test
calls it through the C-ABI twice in a row (the second call finds the first call's leftovers in that array,
with a different query and a smaller budget) and compares each result with bpc_decode_attn on the same inputs.
It is collected last so that a run that stops at the first failure has already run every other test.
"""
import ctypes

import pytest
import torch

from paper_2608_04405_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_context_decode_twice():
    from paper_2608_04405_b200 import binding as B
    from tests import gpu_harness as H
    spec = CONFIGS[1].scaled(n_ctx=6000, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    sess.fit()
    sess.encode()
    units = spec.batch * spec.n_kv_heads
    assert units * sess.w.n_max <= B.lib.bpc_static_scratch_entries()
    P_hash = sess.Ph.to(spec.torch_dtype).contiguous()          # values are already representable: exact
    unit_lens = torch.tensor([sess.lens[u // spec.n_kv_heads] for u in range(units)], dtype=torch.int32, device="cuda")
    tol = H.OUT_TOL[spec.dtype]
    for ppm in (20000, 5000):                                    # second call: other query, shorter index list
        q, _ = sess.w.queries(sess.lens)
        q = q.cuda()
        ref = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=ppm)
        got = B.bpc_decode_attn_static(sess.cfg, q, sess.k_cache, sess.v_cache, sess.codes, P_hash, unit_lens,
                                       budget_ppm=ppm)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert (got - ref).abs().max().item() <= tol
    # and against the CPU checker for one unit, through the regular stage-wise check of the same inputs
    rep = {}
    H.check_decode(sess, q, [1], rep)


def test_static_scratch_rejects_shapes_beyond_its_array():
    from paper_2608_04405_b200 import binding as B
    cfg = B.make_config(4, 32, 8, 131072, 128, torch.bfloat16)   # 4 Mi index entries > 1 Mi
    d = torch.zeros(64, dtype=torch.int64, device="cuda")
    st = B.lib.bpc_decode_attn_static(ctypes.byref(cfg), d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(),
                                      d.data_ptr(), d.data_ptr(), 20000, 0, d.data_ptr(), None)
    assert st == 7                                               # BPC_ERR_SCRATCH_LIMIT, nothing launched
    torch.cuda.synchronize()
