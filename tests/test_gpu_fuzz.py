"""Seeded random shapes through the whole path against the CPU checker: batch, heads per KV head, code length, cache
type, context lengths (ragged, incl. very short), budgets, cluster size, score mode, safeguard, streaming selection,
power-iteration fit, fused and plain steps.
Each case is small enough for the checker to run every stage in full."""
import os
import random

import pytest
import torch

from paper_2608_04405_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as H
    return H


def _cases(n_cases, seed):
    rng = random.Random(seed)
    out = []
    for i in range(n_cases):
        bits = rng.choice([32, 64, 128, 256])
        group = rng.choice([1, 2, 3, 4, 5, 6, 7, 8])
        dtype = rng.choice(["bf16", "bf16", "f32"])
        n_kv = rng.choice([1, 2, 3])
        batch = rng.choice([1, 2, 3])
        n_ctx = rng.choice([64, 300, 1000, 2500, 6000, 12000, 20000])
        ragged = rng.random() < 0.5
        mode = rng.choice([0, 0, 0, 1])
        eas = rng.choice([0, 0, 3000]) if mode == 0 else 0
        cluster = rng.choice([0, 0, 1, 2, 3, 4, 6])
        budget = rng.choice([("ppm", 20000), ("ppm", 1000), ("ppm", 300000), ("count", 1), ("count", 37), ("ppm", 1000000)])
        interleaved = rng.random() < 0.5
        stream = mode == 0 and eas == 0 and rng.random() < 0.3      # streaming selection forced on a shape that would fit
        power = rng.choice([0, 0, 0, 1, 3])                         # power iterations of the fit
        out.append((i, bits, group, dtype, n_kv, batch, n_ctx, ragged, mode, eas, cluster, budget, interleaved, stream, power))
    return out


# more cases or another seed for a one-off run: BPC_FUZZ_CASES, BPC_FUZZ_SEED
@pytest.mark.parametrize("case", _cases(int(os.environ.get("BPC_FUZZ_CASES", "36")), int(os.environ.get("BPC_FUZZ_SEED", "20260811"))),
                         ids=lambda c: "case%d" % c[0])
def test_random_shapes(case, monkeypatch):
    from paper_2608_04405_b200 import binding as B
    H = _harness()
    i, bits, group, dtype, n_kv, batch, n_ctx, ragged, mode, eas, cluster, budget, interleaved, stream, power = case
    stream = bool(stream and mode == 0 and eas == 0)      # the streaming selection covers Hamming scores without the safeguard
    spec = CONFIGS[1].scaled(name="fuzz%d" % i, wid=200 + i, batch=batch, n_kv_heads=n_kv, n_q_heads=n_kv * group, n_ctx=n_ctx,
                             n_ctx_min=max(1, n_ctx // 5) if ragged else None, dtype=dtype, code_bits=bits, steps=2,
                             needles=4, rope_base=None if dtype == "f32" else 500000.0)
    try:
        sess = H.Session(spec, gen_device="cuda", cluster_size=cluster, interleaved=interleaved, score_mode=mode, eas_ppm=eas,
                         fit_power_iters=power, force_streaming=stream)
    except RuntimeError as e:
        if "UNSUPPORTED" in str(e):                     # e.g. a cluster size the shape cannot use
            sess = H.Session(spec, gen_device="cuda", interleaved=interleaved, score_mode=mode, eas_ppm=eas, fit_power_iters=power,
                             force_streaming=stream)
        else:
            raise
    assert sess.ctx.uses_streaming() == stream
    rep = {}
    units = sorted({0, sess.units - 1, sess.units // 2})
    sess.fit(dirty_workspace=True); H.check_fit(sess, units[:1], rep)   # (the workspace holds leftovers)
    sess.encode(); H.check_encode(sess, units, rep, max_keys=4096)
    if eas:
        H.check_eas(sess, units, rep)
    kind, val = budget
    kw = {"budget_ppm": val} if kind == "ppm" else {"budget_count": val}
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), units, rep, **kw)
    k_new, v_new = sess.w.new_kv(sess.lens)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), units, rep, append=(k_new.cuda(), v_new.cuda()), **kw)
    assert sess.ctx.last_device_error() == 0
