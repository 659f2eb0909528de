"""The context-free decode entry point (no allocation inside the library) against the regular one.

Some callers cannot allocate device memory at all - a plug-in in a process whose pool already owns the
device, or code running next to an open stream capture - so they cannot create a library context.  For them
bpc_decode_attn_static keeps its index list and error word in an array built into the library.  This test
calls it through the C-ABI twice in a row (the second call finds the first call's leftovers in that array,
with a different query and a smaller budget) and compares each result with bpc_decode_attn on the same inputs (the two
run the same kernel: bit for bit) and, for the rows that call selected, with the CPU checker's attention.
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
    import numpy as np
    from oracle import bpc_oracle as O
    tol = H.OUT_TOL[spec.dtype]
    G = spec.group
    for ppm in (20000, 5000):                                    # second call: other query, shorter index list
        q, _ = sess.w.queries(sess.lens)
        q = q.cuda()
        sel = torch.full((units, sess.w.n_max), -1, dtype=torch.int32, device="cuda")
        ref = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=ppm, sel_idx=sel)
        got = B.bpc_decode_attn_static(sess.cfg, q, sess.k_cache, sess.v_cache, sess.codes, P_hash, unit_lens,
                                       budget_ppm=ppm)
        torch.cuda.synchronize()
        assert B.bpc_static_last_device_error() == 0
        assert torch.isfinite(got).all()
        assert torch.equal(got, ref), "the context-free call and the context call run the same kernel"
        for u in range(units):                                   # directly against the checker's attention over the selected rows
            bi, h = divmod(u, spec.n_kv_heads)
            n = sess.lens[bi]
            k = O.budget(n, ppm, 0)
            idx = sel[u, :k].cpu().numpy().astype(np.int64)
            want = O.attend(H._np64(q[bi, h * G:(h + 1) * G]), H._np64(sess.k_cache[bi, h, :n]), H._np64(sess.v_cache[bi, h, :n]), idx)
            assert np.abs(want - H._np64(got[bi, h * G:(h + 1) * G])).max() <= tol
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
    cfg32 = B.make_config(1, 4, 1, 4098, 32, torch.bfloat16)     # 32-bit codes need n_max % 4 == 0
    st = B.lib.bpc_decode_attn_static(ctypes.byref(cfg32), d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(),
                                      d.data_ptr(), d.data_ptr(), 20000, 0, d.data_ptr(), None)
    assert st == 1                                               # BPC_ERR_INVALID_ARG
    cfge = B.make_config(1, 4, 1, 4096, 128, torch.bfloat16, eas_ppm=2000)   # the safeguard needs a context
    st = B.lib.bpc_decode_attn_static(ctypes.byref(cfge), d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(),
                                      d.data_ptr(), d.data_ptr(), 20000, 0, d.data_ptr(), None)
    assert st == 2                                               # BPC_ERR_UNSUPPORTED
    torch.cuda.synchronize()
