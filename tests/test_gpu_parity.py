"""GPU parity tests: the CUDA library, called through the C-ABI binding, against the CPU checker."""
import numpy as np
import pytest
import torch

from paper_2608_04405_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as H
    return H


def _decode_loop(sess, steps, units, report, H, check_every=1, fused="alternate"):
    """Decode steps with a cache write each: even steps use bpc_append + bpc_decode_attn, odd steps the fused call."""
    for step in range(steps):
        k_new, v_new = sess.w.new_kv(sess.lens)
        k_new, v_new = k_new.cuda(), v_new.cuda()
        use_fused = fused is True or (fused == "alternate" and step % 2 == 1)
        if use_fused:
            # the query is planted on keys cached before this step, as for the two-call sequence
            q, _ = sess.w.queries(sess.lens, k_cache=sess.k_cache.to(sess.w.device))
            H.check_decode(sess, q.cuda(), units, report, append=(k_new, v_new))
        else:
            H.check_append(sess, k_new, v_new, units, report)
            q, _ = sess.w.queries(sess.lens, k_cache=sess.k_cache.to(sess.w.device))
            if step % check_every == 0:
                H.check_decode(sess, q.cuda(), units, report)


def test_cfg0_tiny_fp32_all_stages():
    """Config 0 exactly: 1 head, n=4096, fp32, 64-bit codes, k=82, 16 decode steps with append."""
    H = _harness()
    spec = CONFIGS[0]
    sess = H.Session(spec)
    rep = {}
    sess.fit(); H.check_fit(sess, [0], rep)
    sess.encode(); H.check_encode(sess, [0], rep)
    _decode_loop(sess, spec.steps, [0], rep, H)
    assert rep["units_checked"] == spec.steps
    print(rep)


@pytest.mark.parametrize("cluster", [1, 2, 3, 4, 5, 6, 7, 8, 9, 12, 16])
def test_cluster_sizes_agree_with_checker(cluster):
    """Ragged length (several tiles plus a tail) at every cluster size, GQA 4, bf16, 128-bit codes."""
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=5000 + 37 * cluster, n_kv_heads=2, n_q_heads=8, steps=2)
    sess = H.Session(spec, cluster_size=cluster)
    rep = {}
    sess.fit(); H.check_fit(sess, [0], rep)
    sess.encode(); H.check_encode(sess, [0, 1], rep)
    _decode_loop(sess, 2, [0, 1], rep, H)
    print(rep)


@pytest.mark.parametrize("bits,group,n,batch", [(128, 4, 5037, 1), (64, 1, 3000, 2), (256, 4, 9000, 1), (128, 7, 20011, 2),
                                                (32, 8, 4000, 1), (128, 2, 70000, 1)])
def test_work_item_kernel_agrees_with_checker(bits, group, n, batch):
    """The alternative decode kernel (persistent grid of work items; selected per context) through the same stage-wise
    checks: decode alone, fused cache write + decode at two consecutive steps, ragged tails, several key ranges."""
    H = _harness()
    spec = CONFIGS[1].scaled(batch=batch, n_ctx=n, n_kv_heads=2, n_q_heads=2 * group, code_bits=bits, steps=2)
    sess = H.Session(spec, gen_device="cuda", decode_path=2, interleaved=(bits == 128))
    assert sess.ctx.uses_work_items()
    rep = {}
    sess.fit()
    sess.encode(); H.check_encode(sess, [0, 1], rep, max_keys=4096)
    units = [0, 2 * batch - 1]
    _decode_loop(sess, 2, units, rep, H)
    q, _ = sess.w.queries(sess.lens, k_cache=sess.k_cache)
    H.check_decode(sess, q, units, rep, budget_ppm=1000000)       # every key selected: dense attention
    H.check_decode(sess, q, units, rep, budget_ppm=0, budget_count=1)
    assert sess.ctx.last_device_error() == 0
    print(rep)


@pytest.mark.parametrize("bits,group,dtype", [(64, 1, "bf16"), (64, 4, "bf16"), (256, 4, "bf16"), (128, 7, "bf16"),
                                              (128, 8, "bf16"), (128, 2, "bf16"), (128, 3, "f32"), (256, 1, "f32"),
                                              (32, 4, "bf16"), (32, 1, "f32"), (32, 8, "bf16")])
def test_code_lengths_and_group_sizes(bits, group, dtype):
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=3000, n_kv_heads=2, n_q_heads=2 * group, code_bits=bits, dtype=dtype, steps=1,
                             rope_base=None if dtype == "f32" else 500000.0)
    sess = H.Session(spec)
    rep = {}
    sess.fit(); H.check_fit(sess, [1], rep)
    sess.encode(); H.check_encode(sess, [0, 1], rep)
    _decode_loop(sess, 2, [0, 1], rep, H)
    print(rep)


@pytest.mark.parametrize("dtype,bits", [("bf16", 128), ("f32", 64)])
def test_interleaved_kv_layout(dtype, bits):
    """K and V rows of a token adjacent in one buffer (row stride 2*head_dim): same results as separate arrays."""
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=4500, n_kv_heads=2, n_q_heads=8, steps=2, dtype=dtype, code_bits=bits)
    sess = H.Session(spec, interleaved=True)
    rep = {}
    sess.fit(); H.check_fit(sess, [1], rep)
    sess.encode(); H.check_encode(sess, [0, 1], rep)
    _decode_loop(sess, 2, [0, 1], rep, H)
    ref = H.Session(spec)
    ref.fit(); ref.encode()
    assert torch.equal(ref.codes[:, :, :4500], sess.codes[:, :, :4500])


@pytest.mark.parametrize("ppm,count", [(1000000, 0), (10000, 0), (50000, 0), (0, 1), (0, 1024), (1, 0)])
def test_budgets(ppm, count):
    """budget = n (dense softmax attention), 1 %, 5 %, a single key, a fixed count, and the smallest fraction."""
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=2500, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    rep = {}
    sess.fit(); sess.encode()
    q, _ = sess.w.queries(sess.lens)
    out, sel = H.check_decode(sess, q.cuda(), [0, 1], rep, budget_ppm=ppm, budget_count=count)
    if ppm == 1000000:
        # every key selected: the result is dense softmax attention
        bi, h = 0, 1
        n = sess.lens[0]
        K = sess.k_cache[bi, h, :n].double().cpu(); V = sess.v_cache[bi, h, :n].double().cpu()
        qq = q[bi, 4:8].double()
        ref = torch.softmax(qq @ K.T / 128 ** 0.5, dim=-1) @ V
        assert (ref - out[bi, 4:8].double().cpu()).abs().max() <= 2e-3


def test_ragged_batch_and_empty_sequence():
    """Different lengths per sequence, one of them empty (output rows are zero, nothing is selected)."""
    H = _harness()
    spec = CONFIGS[3].scaled(batch=3, n_ctx=4000, n_ctx_min=700, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    sess.lens[1] = 0
    sess.ctx.set_seq_lens(sess.lens)
    rep = {}
    sess.fit(); sess.encode()
    lens_q = [max(1, n) for n in sess.lens]
    q, _ = sess.w.queries(lens_q)
    out, sel = H.check_decode(sess, q.cuda(), [0, 1, 4, 5], rep)
    assert torch.count_nonzero(out[1]) == 0
    H.check_encode(sess, [0, 5], rep)


def test_shared_projection_per_kv_head():
    """An externally supplied projection shared by all sequences (offline calibration flow)."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[1].scaled(batch=2, n_ctx=2000, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    sess.fit()
    P_unit = sess.P.clone()
    cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, sess.w.n_max, spec.code_bits, spec.torch_dtype,
                        shared_projection=True)
    ctx2 = B.Context(cfg)
    ctx2.set_seq_lens(sess.lens)
    ctx2.set_projection(P_unit[:spec.n_kv_heads].contiguous())
    sess.ctx, sess.cfg = ctx2, cfg
    sess.P, sess.Ph, sess.gram = ctx2.get_projection()
    sess.codes.zero_()
    rep = {}
    sess.encode(); H.check_encode(sess, [0, 1, 2, 3], rep)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 3], rep)


def test_projection_update_then_decode_without_host_sync():
    """bpc_set_projection and bpc_decode_attn queued back to back on one stream, no host synchronisation between them:
    the decode launch may start early (programmatic dependent launch), but it must hash with the new projection.  The
    context holds another projection until then, so a decode that read P_h too early would select other keys."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="pdl", wid=73, batch=2, n_ctx=6000, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    sess.fit()
    P1 = sess.P.clone()
    P2 = torch.flip(P1, dims=[1]).neg().contiguous()          # the same components, reversed and negated: another valid P
    sess.ctx.set_projection(P2)
    sess.P, sess.Ph, sess.gram = sess.ctx.get_projection()
    sess.encode()                                             # cache codes under P2
    rep = {}
    H.check_encode(sess, [0, 3], rep)
    q, _ = sess.w.queries(sess.lens)
    q = q.cuda()
    filler = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for trial in range(3):
        sess.ctx.set_projection(P1)                           # the context hashes with P1 ...
        torch.cuda.synchronize()

        def switch():
            filler.fill_(trial)                               # (keeps the GPU busy so that the next launches queue up behind it)
            sess.ctx.set_projection(P2)                       # ... until this call, which the decode launch follows directly

        H.check_decode(sess, q, [0, 3], rep, before_decode=switch)


def test_offline_projection_calibration_on_aggregated_keys():
    """Offline Projection Calibration (Section 3.2): Algorithm 1 runs once, ahead of serving, on keys aggregated over
    several sequences (here with two power iterations), one projection per KV head; the serving context takes that
    projection through bpc_set_projection and shares it among all its sequences."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[1].scaled(name="serve", wid=71, batch=3, n_ctx=1500, n_kv_heads=2, n_q_heads=8, steps=1)
    serve = H.Session(spec)
    # calibration context: one "sequence" per KV head holding the keys of all serving sequences of that head
    n_agg = spec.batch * spec.n_ctx
    cal_spec = spec.scaled(name="calib", wid=72, batch=1, n_ctx=n_agg)
    cal = H.Session(cal_spec, fit_power_iters=2)
    for h in range(spec.n_kv_heads):
        cal.k_cache[0, h, :n_agg] = torch.cat([serve.k_cache[b, h, :spec.n_ctx] for b in range(spec.batch)], dim=0)
    rep = {}
    cal.fit(); H.check_fit(cal, [0, 1], rep)
    cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, serve.w.n_max, spec.code_bits, spec.torch_dtype,
                        shared_projection=True)
    ctx2 = B.Context(cfg)
    ctx2.set_seq_lens(serve.lens)
    ctx2.set_projection(cal.P.contiguous())
    serve.ctx, serve.cfg = ctx2, cfg
    serve.P, serve.Ph, serve.gram = ctx2.get_projection()
    serve.encode(); H.check_encode(serve, [0, 3, 5], rep)
    q, _ = serve.w.queries(serve.lens)
    H.check_decode(serve, q.cuda(), [0, 5], rep)
    print(rep)


def test_fused_append_decode_tiny_and_boundary_lengths():
    """Fused cache write at lengths where the new key opens a new chunk / a new 32-key segment, and from n = 0."""
    H = _harness()
    for n0 in (0, 1, 63, 64, 255, 256, 2047):
        spec = CONFIGS[1].scaled(n_ctx=max(n0, 1), n_kv_heads=2, n_q_heads=8, steps=3)
        sess = H.Session(spec, extra_rows=64)
        sess.fit(); sess.encode()            # projection fitted on max(n0, 1) keys
        if n0 == 0:
            sess.lens = [0]
            sess.ctx.set_seq_lens(sess.lens)
        rep = {}
        for step in range(3):
            k_new, v_new = sess.w.new_kv(sess.lens)
            q, _ = sess.w.queries([max(1, n) for n in sess.lens], k_cache=sess.k_cache.to(sess.w.device))
            H.check_decode(sess, q.cuda(), [0, 1], rep, append=(k_new.cuda(), v_new.cuda()), budget_ppm=200000)
        assert sess.lens == [n0 + 3]


@pytest.mark.parametrize("bits,group,dtype,n", [(128, 4, "bf16", 9000), (64, 8, "bf16", 3000), (256, 1, "bf16", 3000),
                                                 (64, 2, "f32", 2500), (128, 3, "bf16", 40000), (32, 4, "bf16", 5000)])
def test_weighted_scores_seven_magnitude_planes(bits, group, dtype, n):
    """Algorithm 3 as printed (sign + 7 magnitude planes per head): scores, selection with the two-level
    histogram, output; separate calls and the fused cache write."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[1].scaled(n_ctx=n, n_kv_heads=2, n_q_heads=2 * group, code_bits=bits, dtype=dtype, steps=2,
                             rope_base=None if dtype == "f32" else 500000.0)
    sess = H.Session(spec, score_mode=B.BPC_SCORE_WEIGHTED7)
    rep = {}
    sess.fit(); sess.encode()
    _decode_loop(sess, 2, [0, 1], rep, H)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 1], rep, budget_ppm=1000000)      # every key selected
    H.check_decode(sess, q.cuda(), [0], rep, budget_ppm=0, budget_count=1)
    print(rep)


@pytest.mark.parametrize("bits,group,n,shift,cluster", [(128, 7, 9000, 0, 0), (128, 8, 20000, 0, 3), (256, 4, 6000, 0, 0),
                                                        (256, 8, 12000, 0, 2), (128, 4, 9000, 2, 0), (64, 8, 7000, 1, 4),
                                                        (128, 7, 40000, 2, 5)])
def test_weighted_scores_wider_than_16_bits(bits, group, n, shift, cluster):
    """Algorithm 3's score where 127 * G * b exceeds 16 bits (seven or eight query heads per KV head at 128 bits: the
    28/4 and 70B-style head layouts; 256-bit codes): the stored keys are shifted right and the keys at the threshold are
    re-scored exactly, so scores, index sets (lowest-index ties) and outputs must equal the checker's as for any other
    shape.  The shift is also forced (diagnostic switch) on shapes that would not need it, where many more keys share a
    stored key and the re-scoring decides most of the ties; several cluster sizes; separate calls and the fused call;
    a dense budget and a single key."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[1].scaled(name="w7wide", wid=70 + group, n_ctx=n, n_kv_heads=2, n_q_heads=2 * group, code_bits=bits, steps=2)
    sess = H.Session(spec, gen_device="cuda", score_mode=B.BPC_SCORE_WEIGHTED7, cluster_size=cluster)
    if shift:
        sess.ctx.debug_force_key_shift(shift)
    rep = {}
    sess.fit(); sess.encode()
    _decode_loop(sess, 2, [0, 1], rep, H)
    q, _ = sess.w.queries(sess.lens)
    for ppm in (1000, 100000, 1000000):
        H.check_decode(sess, q.cuda(), [0, 1], rep, budget_ppm=ppm)
    H.check_decode(sess, q.cuda(), [1], rep, budget_ppm=0, budget_count=1)
    print(rep)


def test_weighted_scores_config4_head_layout_full_size():
    """Configuration 4's shape (28/4 heads: seven query heads per KV head, 128-bit codes, 131072 keys) with the paper's
    weighted score: 127 * 7 * 128 needs 17 bits.  One sequence of the batch at full length, sampled units."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[4].scaled(batch=1, steps=2)
    sess = H.Session(spec, gen_device="cuda", score_mode=B.BPC_SCORE_WEIGHTED7)
    rep = {}
    sess.fit(); sess.encode()
    _decode_loop(sess, 2, [0, 3], rep, H)
    print(rep)


def test_weighted_scores_config2_full_size_fused():
    """The weighted step the benchmark times next to the headline: config 2 at full size (batch 4, clusters of 4),
    cache write fused into the launch, Algorithm 3's score; sampled units."""
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    sess = H.Session(CONFIGS[2].scaled(steps=2), gen_device="cuda", interleaved=True, score_mode=B.BPC_SCORE_WEIGHTED7)
    rep = {}
    sess.fit(); sess.encode()
    _decode_loop(sess, 2, [0, 13, 31], rep, H, fused=True)
    print(sess.ctx.get_cluster_size(), rep)


@pytest.mark.parametrize("bits", [32, 64, 128, 256])
def test_tensor_core_encode_agrees_with_cuda_core_encode(bits):
    """bpc_encode_keys on the tcgen05 path and on the CUDA-core path (diagnostic switch) against each other and
    against the checker: ragged length with a partial last tile, several tiles per block."""
    import os
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=128 * 37 + 5, n_kv_heads=2, n_q_heads=8, code_bits=bits, steps=1)
    sess = H.Session(spec)
    sess.fit()
    sess.encode()                                   # tensor-core path (bf16; 256 bits: two launches)
    tc = sess.codes.clone()
    rep = {}
    H.check_encode(sess, [0, 1], rep)
    sess.ctx.debug_set_tensor_core_encode(False)
    try:
        sess.codes.zero_()
        sess.encode()
    finally:
        sess.ctx.debug_set_tensor_core_encode(True)
    H.check_encode(sess, [0, 1], rep)
    n = sess.lens[0]
    diff = (tc[:, :, :n] != sess.codes[:, :, :n]).any(dim=-1).sum().item()
    # both paths were checked against the fp64 replay above; they may differ from each other only on keys with an
    # ambiguous decision (fp32 tensor-core sums vs fp64 sums), which are rare
    assert diff <= max(2, n // 2000), "%d keys differ between the two encode paths" % diff
    assert torch.count_nonzero(tc[:, :, n:]) == 0   # nothing written past the cached keys


@pytest.mark.parametrize("bits,n", [(128, 70000), (64, 9001), (32, 40000), (256, 20011)])
def test_tensor_core_fit_pass_agrees_with_cuda_core_pass(bits, n):
    """bpc_fit with the pass over the keys on the tensor cores (bf16 caches) and on the CUDA
    cores (diagnostic switch): each against the fp64 replay of Algorithm 1, and the two projections against each other.
    Lengths that are no multiple of the 128-key tile, several blocks per unit, two units of different length."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="fit_tc", wid=74, batch=2, n_ctx=n, n_ctx_min=max(1, n // 3), n_kv_heads=1, n_q_heads=4,
                             code_bits=bits, steps=1)
    sess = H.Session(spec, gen_device="cuda" if n > 20000 else "cpu")
    rep = {}
    sess.fit(dirty_workspace=True)                            # tensor-core pass; the workspace holds leftovers
    H.check_fit(sess, [0, 1], rep)
    err_tc = rep["fit_reconstruction_err_over_K"]
    P_tc, H_tc = sess.P.clone(), [sess.hfit_bits(u) for u in range(2)]
    sess.ctx.debug_set_tensor_core_encode(False)
    try:
        sess.fit(dirty_workspace=True)                        # CUDA-core pass
    finally:
        sess.ctx.debug_set_tensor_core_encode(True)
    rep_cc = {}
    H.check_fit(sess, [0, 1], rep_cc)
    err_cc = rep_cc["fit_reconstruction_err_over_K"]
    # Each run is Algorithm 1 within rounding (checked above), but the two need not agree sign for sign: a decision value
    # inside the rounding band may come out either way, the flipped row moves v_i by 2 K_row / N, and later decisions near
    # zero follow (the more so the longer the code and the shorter the context).  What must agree is the result as a
    # whole: the reconstruction error of the fit, and the leading rows of the projection, found before any such flip.
    for u in range(2):
        rep["rows_differing_u%d" % u] = int((H_tc[u] != sess.hfit_bits(u)).any(axis=1).sum())
    rep["projection_rel_diff"] = ((P_tc - sess.P).norm() / sess.P.norm()).item()
    rep["reconstruction_err"] = (err_tc, err_cc)
    assert abs(err_tc - err_cc) <= 2e-3 * err_cc
    lead = 16
    assert ((P_tc[:, :lead] - sess.P[:, :lead]).norm() / sess.P[:, :lead].norm()).item() <= 1e-3
    print(rep)


def test_error_paths_do_not_launch():
    from paper_2608_04405_b200 import binding as B
    cfg = B.make_config(1, 4, 1, 1024, 128, torch.bfloat16)
    ctx = B.Context(cfg)
    k = torch.zeros(1, 1, 1024, 128, dtype=torch.bfloat16, device="cuda")
    codes = ctx.alloc_codes()
    q = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    before = ctx.launch_count()
    with pytest.raises(B.BpcError) as e:
        ctx.decode_attn(q, k, k, codes)
    assert e.value.status == 4                      # not fitted
    with pytest.raises(B.BpcError) as e:
        ctx.encode_keys(k, codes)
    assert e.value.status == 4
    with pytest.raises(B.BpcError) as e:
        ctx.set_seq_lens([2000])
    assert e.value.status == 3                      # beyond n_max
    ctx.set_projection(torch.randn(1, 128, 128, device="cuda"))
    ctx.set_seq_lens([1024])
    kn = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device="cuda")
    n0 = ctx.launch_count()
    with pytest.raises(B.BpcError) as e:
        ctx.append(kn, kn, k, k, codes)
    assert e.value.status == 3 and ctx.launch_count() == n0      # capacity: nothing launched
    with pytest.raises(B.BpcError) as e:
        ctx.decode_attn(q, k, k, codes, budget_ppm=0, budget_count=0)
    assert e.value.status == 1
    for bad in (dict(code_bits=96), dict(n_q_heads=9), dict(head_dim=64)):
        kw = dict(batch=1, n_q_heads=4, n_kv_heads=1, n_max=1024, code_bits=128, dtype=torch.bfloat16)
        hd = bad.pop("head_dim", 128)
        kw.update(bad)
        with pytest.raises(B.BpcError):
            B.Context(B.make_config(head_dim=hd, **kw))
    assert before == 0


def test_cfg1_full_size_sampled_units():
    """Config 1 at full size (32/8 heads, n=32768, 128-bit codes, k=656): every unit's selection and output."""
    H = _harness()
    spec = CONFIGS[1]
    sess = H.Session(spec, gen_device="cuda")
    rep = {}
    sess.fit(); H.check_fit(sess, [3], rep)
    sess.encode(); H.check_encode(sess, [0, 7], rep, max_keys=8192)
    _decode_loop(sess, 2, list(range(8)), rep, H)
    print(rep)


def test_cfg2_full_size_sampled_units():
    """Config 2 at full size (batch 4, n=131072) in the launch configuration the benchmark times; sampled units."""
    H = _harness()
    spec = CONFIGS[2]
    sess = H.Session(spec, gen_device="cuda")
    rep = {}
    sess.fit()
    sess.encode(); H.check_encode(sess, [5], rep, key_slice=(120000, 124096))
    # two steps: bpc_append + bpc_decode_attn, then the fused bpc_append_decode_attn launch (the one the benchmark times)
    _decode_loop(sess, 2, [0, 13, 31], rep, H)
    # planted-needle recall of the selection is the same number on both sides because the index sets are identical
    print(rep)


@pytest.mark.parametrize("bits", [64, 128, 256])
def test_cfg3_ragged_sweep_code_length_and_budget(bits):
    """Config 3's sweep (code length x budget) on a ragged batch with lengths in [16384, 65536]; batch reduced to 4,
    the full-batch launch geometry is covered by the next test."""
    H = _harness()
    spec = CONFIGS[3].scaled(batch=4, code_bits=bits, steps=2)
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    rep = {}
    sess.fit()
    sess.encode(); H.check_encode(sess, [3], rep, max_keys=4096)
    q, _ = sess.w.queries(sess.lens)
    for ppm in (10000, 20000, 50000):
        H.check_decode(sess, q.cuda(), [1, 30], rep, budget_ppm=ppm)
    k_new, v_new = sess.w.new_kv(sess.lens)
    H.check_decode(sess, q.cuda(), [9, 22], rep, append=(k_new.cuda(), v_new.cuda()))
    print(sess.lens, rep)


@pytest.mark.parametrize("bits", [64, 128, 256])
def test_cfg3_full_batch_sampled_units(bits):
    """Config 3 at full size (batch 16, 128 units, one block per unit) in the benchmark's launch configuration, at the
    three code lengths of its sweep: the fit and the encode of one unit each (at 256 bits the encode is two launches),
    then fused decode steps."""
    H = _harness()
    spec = CONFIGS[3].scaled(code_bits=bits)
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    rep = {}
    sess.fit(dirty_workspace=True); H.check_fit(sess, [41], rep)
    sess.encode(); H.check_encode(sess, [100], rep, max_keys=4096)
    _decode_loop(sess, 2, [0, 77, 127], rep, H, fused=True)
    print(sess.ctx.get_cluster_size(), rep)


def test_cfg4_full_size_sampled_units():
    """Config 4 at full size (batch 8, 28/4 heads: 7 query heads per KV head, n = 131072): prefill fit + encode, then
    fused decode steps; sampled units."""
    H = _harness()
    spec = CONFIGS[4]
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    rep = {}
    sess.fit(); H.check_fit(sess, [17], rep)
    sess.encode(); H.check_encode(sess, [2, 31], rep, key_slice=(60000, 64096))
    _decode_loop(sess, 2, [0, 19, 31], rep, H, fused=True)
    print(rep)


@pytest.mark.parametrize("dtype,bits,n,power", [("bf16", 128, 20000, 2), ("f32", 64, 9000, 1), ("bf16", 64, 70000, 4)])
def test_fit_with_power_iterations(dtype, bits, n, power):
    """bpc_fit with cfg.fit_power_iters = n: the binary component of every bit is sign((R R^T)^n R v*^T) (section "Binary
    Principal Components Finding"); replayed by the checker with the library's signs adopted inside the fp32 ambiguity
    band, then the usual encode and decode checks on the projection it produced."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="powerfit", wid=60 + power, batch=2, n_q_heads=8, n_kv_heads=2, n_ctx=n, dtype=dtype,
                             code_bits=bits, steps=2)
    sess = H.Session(spec, gen_device="cuda", fit_power_iters=power)
    rep = {}
    sess.fit(); H.check_fit(sess, [0, 3], rep)
    sess.encode(); H.check_encode(sess, [1], rep, max_keys=4096)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 3], rep)
    print(rep)


def test_streaming_selection_two_million_keys():
    """A unit longer than the largest cluster's shared memory holds with 16-bit score keys (the 2M-token point of the
    paper's latency-vs-context study).  The library takes byte keys there when the scores allow it (checked first); with
    those ruled out it switches to the streaming selection (per-warp histograms, codes read twice), which is what shapes
    with more than 256 distinct scores get.  Same checks as everywhere else, on a 2-KV-head model to bound memory: plain
    and fused steps, fixed budget of 2048 keys."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="stream2m", wid=90, batch=1, n_kv_heads=2, n_q_heads=8, n_ctx=2097152, code_bits=64, steps=2)
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    assert sess.ctx.uses_byte_keys() and not sess.ctx.uses_streaming()
    rep = {}
    sess.fit()
    sess.encode()
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 1], rep, budget_count=2048)              # byte keys, the library's own choice
    sess.ctx.debug_force_byte_keys(-1)
    assert sess.ctx.uses_streaming()
    sess.fit()
    sess.encode(); H.check_encode(sess, [1], rep, max_keys=4096)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 1], rep, budget_count=2048)
    k_new, v_new = sess.w.new_kv(sess.lens)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [1], rep, budget_count=1024, append=(k_new.cuda(), v_new.cuda()))
    print(rep)


@pytest.mark.parametrize("dtype,bits,group,n,cluster", [("bf16", 128, 4, 40000, 4), ("f32", 64, 2, 9000, 2), ("bf16", 256, 8, 7000, 1),
                                                        ("bf16", 32, 4, 12000, 2)])
def test_streaming_selection_forced_at_ordinary_sizes(dtype, bits, group, n, cluster):
    """The streaming selection forced on contexts that would fit (diagnostic switch), so that it is checked stage by
    stage at sizes the checker handles in full: several cluster sizes, both cache types, fused steps and ties."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="streamf", wid=91 + group, batch=2, n_kv_heads=2, n_q_heads=2 * group, n_ctx=n, dtype=dtype,
                             code_bits=bits, steps=3)
    sess = H.Session(spec, gen_device="cuda", cluster_size=cluster, force_streaming=True)
    assert sess.ctx.uses_streaming()
    rep = {}
    sess.fit(); sess.encode()
    _decode_loop(sess, 3, [0, 3], rep, H)
    q, _ = sess.w.queries(sess.lens)
    for ppm in (1000, 500000, 1000000):
        H.check_decode(sess, q.cuda(), [1, 2], rep, budget_ppm=ppm)
    print(rep)


def test_selection_variant_switched_on_a_live_context():
    """The diagnostic switch between the in-shared-memory and the streaming selection on a context that has already
    launched the other variant (each variant is its own kernel, with function attributes of its own)."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="switch", wid=75, n_ctx=30000, n_kv_heads=2, n_q_heads=8, steps=1)
    sess = H.Session(spec)
    rep = {}
    sess.fit(); sess.encode()
    q, _ = sess.w.queries(sess.lens)
    q = q.cuda()
    H.check_decode(sess, q, [0, 1], rep)
    for on in (True, False, True):
        sess.ctx.debug_force_streaming(on)
        assert sess.ctx.uses_streaming() == on
        H.check_decode(sess, q, [0, 1], rep)


@pytest.mark.parametrize("dtype,bits,group,n", [("bf16", 128, 4, 9000), ("f32", 64, 2, 5000), ("bf16", 256, 8, 6000), ("bf16", 32, 4, 7000)])
def test_quality_yardsticks(dtype, bits, group, n):
    """The TOPK (Oracle) selector and dense attention (appendix "Baseline Methods"; cosine-similarity table), and the two
    numbers built on them: recall of the hash selection against the exact top-k, cosine of sparse against dense output."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="yard", wid=80 + group, batch=2, n_kv_heads=2, n_q_heads=2 * group, n_ctx=n, dtype=dtype,
                             code_bits=bits, steps=1)
    sess = H.Session(spec, gen_device="cuda")
    rep = {}
    sess.fit(); sess.encode()
    q, _ = sess.w.queries(sess.lens)
    H.check_yardsticks(sess, q.cuda(), [0, 3], rep)
    H.check_yardsticks(sess, q.cuda(), [1], rep, budget_ppm=100000)
    print(rep)


@pytest.mark.parametrize("n_ctx,batch", [(262144, 1), (32768, 16), (131072, 3)])
def test_sweep_shapes_single_word_codes_fixed_budgets(n_ctx, batch):
    """The second bench workload's shapes (Section 4 "Setup" / latency-vs-context study: 64-bit codes, budgets of 1024
    and 2048 keys) at full size in the launch geometry the sweep times: long context at batch 1 (cluster size 10),
    short context at batch 16 (cluster size 1), and a batch that is not a power of two (24 units, cluster size 5);
    sampled units, plain and fused steps."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="sweep", wid=40 + batch, batch=batch, n_ctx=n_ctx, code_bits=64, steps=2)
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    rep = {}
    sess.fit()
    sess.encode(); H.check_encode(sess, [2], rep, max_keys=4096)
    units = [0, sess.units - 1]
    for budget in (1024, 2048):
        q, _ = sess.w.queries(sess.lens)
        H.check_decode(sess, q.cuda(), units, rep, budget_count=budget)
    k_new, v_new = sess.w.new_kv(sess.lens)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), units, rep, budget_count=2048, append=(k_new.cuda(), v_new.cuda()))
    print(rep)


@pytest.mark.parametrize("dtype,bits,group,n,batch,cluster", [("bf16", 64, 4, 30011, 2, 0), ("bf16", 64, 1, 9000, 1, 3), ("bf16", 32, 4, 20000, 1, 0),
                                                              ("bf16", 128, 2, 9000, 2, 1), ("f32", 64, 2, 6000, 1, 2), ("bf16", 32, 7, 4097, 1, 5)])
def test_byte_score_keys_forced_at_ordinary_sizes(dtype, bits, group, n, batch, cluster):
    """Kernel variant with byte score keys (Hamming scores with at most 256 distinct values), forced at ordinary sizes:
    against the checker stage by stage, plain and fused steps, and bit for bit against the 16-bit-key variant."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="k8", wid=76, batch=batch, n_ctx=n, n_ctx_min=max(1, n // 2) if batch > 1 else None, n_kv_heads=2,
                             n_q_heads=2 * group, code_bits=bits, dtype=dtype, steps=2, rope_base=None if dtype == "f32" else 500000.0)
    sess = H.Session(spec, cluster_size=cluster)
    rep = {}
    sess.fit(); sess.encode()
    q, _ = sess.w.queries(sess.lens)
    q = q.cuda()
    units = [0, sess.units - 1]
    ref = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=20000).clone()
    sess.ctx.debug_force_byte_keys(1)
    assert sess.ctx.uses_byte_keys()
    if cluster:
        sess.ctx.set_cluster_size(cluster)
    for ppm, count in ((20000, 0), (1000000, 0), (0, 7)):
        H.check_decode(sess, q, units, rep, budget_ppm=ppm, budget_count=count)
    got = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=20000)
    torch.cuda.synchronize()
    assert torch.equal(got, ref), "byte keys and 16-bit keys select and attend the same rows"
    k_new, v_new = sess.w.new_kv(sess.lens)
    H.check_decode(sess, q, units, rep, append=(k_new.cuda(), v_new.cuda()))
    sess.ctx.debug_force_byte_keys(-1)
    assert not sess.ctx.uses_byte_keys()
    print(rep)


def test_byte_score_keys_are_refused_where_scores_need_more_than_a_byte():
    H = _harness()
    from paper_2608_04405_b200 import binding as B
    spec = CONFIGS[1].scaled(name="k8no", wid=77, n_ctx=4000, n_kv_heads=2, n_q_heads=16, code_bits=64, steps=1)   # 8 heads x 64 bits / 2 = 256
    sess = H.Session(spec)
    with pytest.raises(B.BpcError) as e:
        sess.ctx.debug_force_byte_keys(1)
    assert e.value.status == 2                                   # BPC_ERR_UNSUPPORTED
    assert not sess.ctx.uses_byte_keys()


def test_million_key_context_takes_byte_keys_by_itself():
    """One million keys per unit at batch 1 (8 units, 64-bit codes): with 16-bit keys a unit needs 16 blocks, of which
    only 7 clusters are resident at once; the library takes byte keys and clusters that run in one wave."""
    H = _harness()
    spec = CONFIGS[1].scaled(name="mega", wid=78, batch=1, n_ctx=1048576, code_bits=64, steps=2)
    sess = H.Session(spec, gen_device="cuda", interleaved=True)
    assert sess.ctx.uses_byte_keys() and not sess.ctx.uses_streaming()
    rep = {}
    sess.fit(); sess.encode()
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 7], rep, budget_count=2048)
    k_new, v_new = sess.w.new_kv(sess.lens)
    H.check_decode(sess, q.cuda(), [3], rep, budget_count=1024, append=(k_new.cuda(), v_new.cuda()))
    print(sess.ctx.get_cluster_size(), rep)


@pytest.mark.parametrize("dtype,bits,group,n,cluster", [("bf16", 128, 4, 9000, 0), ("bf16", 128, 4, 9000, 1), ("bf16", 64, 8, 5000, 2),
                                                        ("f32", 64, 2, 4096, 0), ("bf16", 256, 1, 3000, 0), ("bf16", 32, 4, 6000, 0)])
def test_error_aware_safeguard(dtype, bits, group, n, cluster):
    """EAS: per-key reconstruction errors from both encode paths, the static hard-to-hash set, and decode steps whose
    selection is the union of the hash top-(k - m) and that set (10 % of a 2 % budget), incl. the fused cache write."""
    H = _harness()
    spec = CONFIGS[1].scaled(n_ctx=n, n_kv_heads=2, n_q_heads=2 * group, code_bits=bits, dtype=dtype, steps=2,
                             rope_base=None if dtype == "f32" else 500000.0)
    sess = H.Session(spec, eas_ppm=2000, cluster_size=cluster)
    rep = {}
    sess.fit(); sess.encode()
    H.check_eas(sess, [0, 1], rep)
    _decode_loop(sess, 2, [0, 1], rep, H)
    q, _ = sess.w.queries(sess.lens)
    H.check_decode(sess, q.cuda(), [0, 1], rep, budget_ppm=0, budget_count=5)          # budget below the set size
    H.check_decode(sess, q.cuda(), [0, 1], rep, budget_ppm=1000000)                    # everything: all duplicates
    H.check_decode(sess, q.cuda(), [1], rep, budget_ppm=500000)
    print(rep)


def test_error_aware_safeguard_full_size_cfg2():
    H = _harness()
    spec = CONFIGS[2].scaled(batch=2)
    sess = H.Session(spec, gen_device="cuda", interleaved=True, eas_ppm=2000)
    rep = {}
    sess.fit(); sess.encode()
    H.check_eas(sess, [3, 12], rep)
    _decode_loop(sess, 2, [3, 12, 15], rep, H, fused=True)
    print(rep)
