"""Stage-wise comparison of the CUDA library (through the C-ABI binding) with the CPU checker.

Every stage is checked on the same seeded inputs, and each downstream stage is additionally fed the
library's own upstream output (its projection, its codes, its index set), so that a legitimately ambiguous
sign upstream cannot masquerade as a downstream bug.

Tolerances
  fit      : a fitted sign may differ only where |t| < 1e-5 * ||r|| * ||v*|| (fp32 row dot product);
             with the library's signs adopted, P must agree to 2e-5 relative per row
  encode   : bits bit-exact except decisions with |t| < 1e-6 * (||k|| ||P_i|| + sum_{j<i} |G_ji|), counted
  query    : collapsed weights exact except bits with |p_j| < 1e-6 * ||q|| * ||P_j||, counted
  scores   : bit-exact given the library's codes and query weights
  top-k    : index set bit-exact (ascending, lowest-index ties)
  output   : max-abs 2e-3 (bf16 caches) / 1e-5 (fp32 caches) against the fp64 checker
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import bpc_oracle as O
from paper_2608_04405_b200 import binding as B
from paper_2608_04405_b200.inputs import Workload, WorkloadSpec

OUT_TOL = {"bf16": 2e-3, "f32": 1e-5}


def _np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def codes_to_bits(codes_unit: torch.Tensor, b: int) -> np.ndarray:
    """codes [n, b/64] int64 (or [n, 1] int32 at b = 32; device or host) -> bits [n, b] uint8."""
    if b == 32:          # widen the 32-bit words to the 64-bit words the checker unpacks (upper half zero)
        w = codes_unit.detach().cpu().numpy().view(np.uint32).astype(np.uint64)
        return O.unpack_bits(w, b)
    w = codes_unit.detach().cpu().numpy().view(np.uint64)
    return O.unpack_bits(w, b)


class Session:
    """A workload on the GPU with its library context, fitted and encoded."""

    def __init__(self, spec: WorkloadSpec, gen_device: str = "cpu", salt: int = 0, cluster_size: int = 0,
                 extra_rows=None, interleaved: bool = False, score_mode: int = 0, eas_ppm: int = 0, fit_power_iters: int = 0,
                 decode_path: int = 0, force_streaming: bool = False):
        self.spec = spec
        self.w = Workload(spec, device=gen_device, extra_rows=extra_rows, salt=salt)
        dev = "cuda"
        if interleaved:       # K and V rows of a token adjacent in one buffer; the caches are strided views of it
            self.kv_buf, self.k_cache, self.v_cache = B.interleaved_kv(spec.batch, spec.n_kv_heads, self.w.n_max,
                                                                        spec.head_dim, spec.torch_dtype)
            self.k_cache.copy_(self.w.k_cache)
            self.v_cache.copy_(self.w.v_cache)
        else:
            self.k_cache = self.w.k_cache.to(dev)
            self.v_cache = self.w.v_cache.to(dev)
        self.v_star = self.w.v_star.to(dev)
        self.cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, self.w.n_max, spec.code_bits,
                                 spec.torch_dtype, kv_row_stride=2 * spec.head_dim if interleaved else 0,
                                 score_mode=score_mode, eas_ppm=eas_ppm, fit_power_iters=fit_power_iters)
        self.s_err = None
        self.ctx = B.Context(self.cfg)
        if force_streaming:
            self.ctx.debug_force_streaming(True)
        if cluster_size:
            self.ctx.set_cluster_size(cluster_size)
        if decode_path:
            self.ctx.debug_set_decode_path(decode_path)
        self.lens = list(self.w.seq_lens)
        self.ctx.set_seq_lens(self.lens)
        self.codes = self.ctx.alloc_codes()
        self.units = spec.batch * spec.n_kv_heads
        self.fit_ws = None

    def fit(self, dirty_workspace: bool = False):
        """dirty_workspace: hand bpc_fit a workspace full of ones (the library must not rely on its contents)."""
        self.fit_ws = torch.full((self.ctx.fit_workspace_bytes(),), 255 if dirty_workspace else 0, dtype=torch.uint8, device="cuda")
        self.ctx.fit(self.k_cache, self.v_star, self.fit_ws)
        torch.cuda.synchronize()
        self.P, self.Ph, self.gram = self.ctx.get_projection()
        torch.cuda.synchronize()

    def encode(self):
        self.ctx.encode_keys(self.k_cache, self.codes)
        torch.cuda.synchronize()

    def unit_views(self, u: int):
        s = self.spec
        bi, h = divmod(u, s.n_kv_heads)
        return bi, h, self.lens[bi]

    def hfit_bits(self, u: int) -> np.ndarray:
        s = self.spec
        off = self.ctx.fit_codes_offset()
        if s.code_bits == 32:
            raw = self.fit_ws[off: off + self.units * self.w.n_max * 4].view(torch.int32).view(self.units, self.w.n_max, 1)
            _, _, n = self.unit_views(u)
            return codes_to_bits(raw[u, :n], 32)
        words = s.code_bits // 64
        n_max = self.w.n_max
        raw = self.fit_ws[off: off + self.units * n_max * words * 8].view(torch.int64).view(self.units, n_max, words)
        _, _, n = self.unit_views(u)
        return codes_to_bits(raw[u, :n], s.code_bits)


def check_fit(sess: Session, units, report: dict):
    s = sess.spec
    for u in units:
        bi, h, n = sess.unit_views(u)
        K = _np64(sess.k_cache[bi, h, :n])
        vs = _np64(sess.v_star[u])
        gpuH = sess.hfit_bits(u)
        gpuP = _np64(sess.P[u])
        # replay Algorithm 1 in fp64, adopting the library's signs where the decision is within fp32 noise.  The
        # library never stores the residual: it forms t = K_row.d - sum_{j<i} u_j (v_j.d) from fp32 partial sums, so its
        # rounding error scales with |K_row||d| + sum_j |v_j.d| (not with the residual): that bound, 32 * 2^-24 of
        # those magnitudes, is part of the band inside which a sign may differ, next to 1e-5 |r||d|.
        R = K.copy()
        amb = hard = 0
        Pref = np.zeros_like(gpuP)
        npow = int(sess.cfg.fit_power_iters)
        Knorm = np.linalg.norm(K, axis=1)
        eps_band = 32.0 * 2.0 ** -24
        K_energy = float((K * K).sum())
        for i in range(s.code_bits):
            z = vs[i].copy()                                 # direction: v*, or (R^T R)^n v* for the power-iteration fit
            for _ in range(npow):
                z = R.T @ (R @ z)
                z = z / max(np.linalg.norm(z), 1e-300)
            t = R @ z
            mine = t >= 0
            theirs = gpuH[:, i].astype(bool)
            diff = mine != theirs
            tau = 1e-5 * np.linalg.norm(R, axis=1) * np.linalg.norm(z) + \
                eps_band * (Knorm * np.linalg.norm(z) + float(np.abs(Pref[:i] @ z).sum()))
            if npow > 0:
                # the library's R^T R is the keys' Gram matrix minus the rank-one terms N v^T v (v rounded to fp32): its
                # absolute error is about 4 * 2^-24 |K|_F^2, so the direction (R^T R)^n v* is off by about n times that
                # over the largest eigenvalue of R^T R, which exceeds 1 once the residual has all but vanished
                lam = float(np.linalg.norm(R.T @ R, 2))
                kappa = npow * 4.0 * 2.0 ** -24 * K_energy / max(lam, 1e-300)
                tau = tau + min(kappa, 1e6) * np.linalg.norm(R, axis=1) * np.linalg.norm(z)
            hard += int(np.count_nonzero(diff & (np.abs(t) >= tau)))
            amb += int(np.count_nonzero(diff & (np.abs(t) < tau)))
            uu = np.where(theirs, 1.0, -1.0)
            v = (uu @ R) / n
            R = R - np.outer(uu, v)
            Pref[i] = v
        assert hard == 0, "fit: %d sign decisions differ outside the ambiguity band (unit %d)" % (hard, u)
        # Whatever signs were adopted inside the band (which is wide once the residual has all but vanished, e.g. for a
        # context shorter than the code length, or where the power iteration's tracked Gram matrix holds only rounding
        # noise), the library's own pair (H, P) must reconstruct the keys as well as the fp64 replay of those signs does:
        # || K - H P ||_F <= || R_b ||_F + 2e-5 * sqrt(b) * || K ||_F (the row tolerance below, summed over the b rows).
        # Where the residual has vanished this pins the reconstruction at rounding level.
        Hpm = 2.0 * gpuH.astype(np.float64) - 1.0
        rec_err = float(np.linalg.norm(K - Hpm @ gpuP))
        bound = float(np.linalg.norm(R)) * (1.0 + 1e-3) + 2e-5 * np.sqrt(s.code_bits) * float(np.linalg.norm(K))
        assert rec_err <= bound, "fit: || K - H P ||_F = %g exceeds the replayed residual %g (unit %d)" % (rec_err, bound, u)
        report["fit_reconstruction_err_over_K"] = max(report.get("fit_reconstruction_err_over_K", 0.0),
                                                      rec_err / max(float(np.linalg.norm(K)), 1e-300))
        # rows: 2e-5 relative, plus the same absolute rounding floor in units of a typical key row (a row of P that is
        # itself at rounding level, e.g. once the residual of a tiny context has vanished, cannot be held to 2e-5 of itself)
        floor = eps_band * float(np.linalg.norm(K) / np.sqrt(max(n, 1)))
        rel = (np.linalg.norm(gpuP - Pref, axis=1) - floor) / np.maximum(np.linalg.norm(Pref, axis=1), 1e-30)
        assert rel.max() <= 2e-5, "fit: projection rows differ, max relative error %g (unit %d)" % (rel.max(), u)
        # P_h is P rounded to the cache precision; Gram = P_h P_h^T
        Ph = O.to_hash_precision(_np64(sess.P[u]), s.dtype)
        assert np.array_equal(Ph, _np64(sess.Ph[u])), "hash-precision rounding of P differs"
        Gm = Ph @ Ph.T
        gerr = np.abs(_np64(sess.gram[u]) - Gm).max() / max(np.abs(Gm).max(), 1e-30)
        assert gerr <= 1e-6, "Gram matrix differs (%g)" % gerr
        report["fit_ambiguous_signs"] = report.get("fit_ambiguous_signs", 0) + amb
        report["fit_max_rel_err"] = max(report.get("fit_max_rel_err", 0.0), float(max(rel.max(), 0.0)))
        # pure-checker fit from scratch agrees wherever no sign was ambiguous
        if amb == 0:
            P0, _, _ = O.fit(K, vs, power_iters=npow)
            rel0 = (np.linalg.norm(gpuP - P0, axis=1) - floor) / np.maximum(np.linalg.norm(P0, axis=1), 1e-30)
            assert rel0.max() <= 2e-5


def check_encode(sess: Session, units, report: dict, max_keys: int = 0, key_slice=None):
    s = sess.spec
    for u in units:
        bi, h, n = sess.unit_views(u)
        lo, hi = (0, n) if key_slice is None else key_slice
        if max_keys and hi - lo > max_keys:
            hi = lo + max_keys
        K = _np64(sess.k_cache[bi, h, lo:hi])
        Ph = _np64(sess.Ph[u if sess.cfg.hash_sets == sess.units else h])
        bits = codes_to_bits(sess.codes[bi, h, lo:hi], s.code_bits)
        hard, amb = O.replay_encode_with_adoption(K, Ph, bits)
        assert not hard.any(), "encode: %d bits differ outside the ambiguity band (unit %d)" % (int(hard.sum()), u)
        report["encode_ambiguous_bits"] = report.get("encode_ambiguous_bits", 0) + int(amb.sum())
        report["encode_bits_checked"] = report.get("encode_bits_checked", 0) + int(bits.size)
        if not amb.any():
            ref, _ = O.encode(K, Ph)
            assert np.array_equal(ref, bits)


def check_eas(sess: Session, units, report: dict):
    """bpc_build_eas: squared reconstruction errors (Eq. 8) against the fp64 residual norms, and the hard-to-hash set
    as a valid top-m of them (keys whose errors differ by less than the fp32 noise of the sweep may swap)."""
    s = sess.spec
    sess.ctx.build_eas()
    torch.cuda.synchronize()
    err, idx, cnt = sess.ctx.get_eas()
    torch.cuda.synchronize()
    sess.s_err = [idx[u, :int(cnt[u])].cpu().numpy().astype(np.int64) for u in range(sess.units)]
    for u in units:
        bi, h, n = sess.unit_views(u)
        K = _np64(sess.k_cache[bi, h, :n])
        Ph = _np64(sess.Ph[u if sess.cfg.hash_sets == sess.units else h])
        bits = codes_to_bits(sess.codes[bi, h, :n], s.code_bits)
        ref = np.linalg.norm(K - (2.0 * bits - 1.0) @ Ph, axis=1) ** 2          # from the library's own codes
        got = err[u, :n].double().cpu().numpy()
        scale = (np.linalg.norm(K, axis=1) ** 2).max()
        assert np.abs(got - ref).max() <= 2e-5 * scale, "squared reconstruction errors differ: %g" % np.abs(got - ref).max()
        m = -(-n * sess.cfg.eas_ppm // 1000000)
        mine = sess.s_err[u]
        assert len(mine) == m and np.all(np.diff(mine) > 0) and (len(mine) == 0 or (mine[0] >= 0 and mine[-1] < n))
        # exactly the top-m of the library's own error values, ties to the lowest index
        assert np.array_equal(mine, O.eas_set(got, m)), "hard-to-hash set is not the top-m of the recorded errors"
        # and a valid top-m of the fp64 errors up to the fp32 noise
        thr = np.sort(ref)[::-1][m - 1] if m > 0 else np.inf
        tol = 4e-5 * scale
        assert np.all(ref[mine] >= thr - tol)
        rest = np.setdiff1d(np.arange(n), mine)
        assert np.all(ref[rest] <= thr + tol)
        report["eas_keys"] = report.get("eas_keys", 0) + m


def check_decode(sess: Session, q: torch.Tensor, units, report: dict, budget_ppm=None, budget_count=0, append=None,
                 before_decode=None):
    """One decode step through the library, checked stage by stage for the given units.

    With append=(k_new, v_new) the step goes through the fused bpc_append_decode_attn call; the cache rows, the
    new key's code and the advanced lengths are checked as for bpc_append, and the plain decode call that
    follows must reproduce the fused call's output bit for bit.  before_decode, if given, is called right before the
    decode call with no host synchronisation in between (work it queues on the stream precedes the decode launch)."""
    s = sess.spec
    ppm = s.budget_ppm if budget_ppm is None else budget_ppm
    n_max = sess.w.n_max
    dbg_scores = torch.zeros(sess.units, n_max, dtype=torch.int32, device="cuda")
    dbg_qw = torch.zeros(sess.units, s.code_bits, dtype=torch.int32, device="cuda")
    sel = torch.full((sess.units, n_max), -1, dtype=torch.int32, device="cuda")
    sess.ctx.debug_set_buffers(dbg_scores, dbg_qw)
    if before_decode is not None:
        before_decode()
    if append is None:
        out = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=ppm, budget_count=budget_count,
                                   sel_idx=sel)
    else:
        k_new, v_new = append
        out = sess.ctx.append_decode_attn(k_new, v_new, sess.k_cache, sess.v_cache, sess.codes, q, budget_ppm=ppm,
                                          budget_count=budget_count, sel_idx=sel)
    torch.cuda.synchronize()
    sess.ctx.debug_set_buffers(None, None)
    assert sess.ctx.last_device_error() == 0
    if append is not None:
        sess.lens = [n + 1 for n in sess.lens]
        assert sess.ctx.get_seq_lens() == sess.lens
        for u in units:
            bi, h, n1 = sess.unit_views(u)
            assert torch.equal(sess.k_cache[bi, h, n1 - 1], k_new[bi, h]) and torch.equal(sess.v_cache[bi, h, n1 - 1], v_new[bi, h])
            check_encode(sess, [u], report, key_slice=(n1 - 1, n1))
    # a second call without the parity buffers and without a caller index list must give the same output
    out2 = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=ppm, budget_count=budget_count)
    torch.cuda.synchronize()
    if sess.s_err is not None and append is not None:
        # with a safeguard set every block also attends the safeguard keys of its own key range, and the fused call
        # splits the key range differently (the appending block takes a smaller share): same rows, another summation order
        assert (out - out2).abs().max().item() <= 1e-5, "fused and plain decode disagree"
    else:
        assert torch.equal(out, out2), "decode is not reproducible between calls"
    G = s.group
    tol = OUT_TOL[s.dtype]
    for u in units:
        bi, h, n = sess.unit_views(u)
        Ph = _np64(sess.Ph[u if sess.cfg.hash_sets == sess.units else h])
        qg = _np64(q[bi, h * G:(h + 1) * G])
        K = _np64(sess.k_cache[bi, h, :n])
        V = _np64(sess.v_cache[bi, h, :n])
        bits = codes_to_bits(sess.codes[bi, h, :n], s.code_bits)
        # query hash
        mode = O.WEIGHTED7 if sess.cfg.score_mode == B.BPC_SCORE_WEIGHTED7 else O.HAMMING
        p, sg, a = O.query_hash(qg, Ph, mode)
        A = O.collapsed_weights(sg, a)
        A_gpu = dbg_qw[u].cpu().numpy().astype(np.int64)
        if not np.array_equal(A, A_gpu):
            band = np.stack([O.ambiguity_threshold_query(qg[g], Ph) for g in range(G)])
            amb_bits = np.abs(p) < band
            # flipping only ambiguous head signs must be able to explain the difference
            slack = 2 * (amb_bits * a).sum(axis=0)
            if mode == O.WEIGHTED7:
                # ... or a magnitude that sits on a rounding boundary of the 7-bit quantiser (one step per head)
                frac = 127.0 * np.abs(p) / np.maximum(np.abs(p).max(axis=1, keepdims=True), 1e-300)
                slack = slack + (np.abs(frac - np.floor(frac) - 0.5) < 1e-4).sum(axis=0)
            assert np.all(np.abs(A - A_gpu) <= slack), "query hash differs outside the ambiguity band (unit %d)" % u
            report["query_ambiguous_bits"] = report.get("query_ambiguous_bits", 0) + int(np.count_nonzero(A != A_gpu))
        # scores from the library's codes and the library's query weights
        hpm = 2 * bits.astype(np.int64) - 1
        sc = hpm @ A_gpu
        sc_gpu = dbg_scores[u, :n].cpu().numpy().astype(np.int64)
        assert np.array_equal(sc, sc_gpu), "hash scores differ (unit %d): %d of %d" % (u, int((sc != sc_gpu).sum()), n)
        if np.array_equal(A, A_gpu):
            assert np.array_equal(O.hash_scores(bits, sg, a), sc_gpu)
        # selection
        k = O.budget(n, ppm, budget_count)
        if sess.s_err is None:
            idx = O.topk(sc_gpu, k)
            idx_gpu = sel[u, :k].cpu().numpy().astype(np.int64)
            assert np.array_equal(idx, idx_gpu), "selected index set differs (unit %d)" % u
        else:
            # error-aware safeguard: k - me hash-selected keys, then the first me safeguard keys with -1 for duplicates
            s_err = sess.s_err[u]
            me = min(len(s_err), k)
            hash_idx = O.topk(sc_gpu, k - me)
            got_hash = sel[u, :k - me].cpu().numpy().astype(np.int64)
            assert np.array_equal(hash_idx, got_hash), "hash-selected part differs (unit %d)" % u
            want_tail = np.where(np.isin(s_err[:me], hash_idx), -1, s_err[:me])
            got_tail = sel[u, k - me:k].cpu().numpy().astype(np.int64)
            assert np.array_equal(want_tail, got_tail), "safeguard part of the index list differs (unit %d)" % u
            idx_gpu = O.eas_union(hash_idx, s_err[:me])
            ref_unit = O.decode_unit(qg, K, V, bits, Ph, ppm, budget_count, mode=mode, s_err=s_err)
            if np.array_equal(A, A_gpu):
                assert np.array_equal(ref_unit["idx"], idx_gpu)
        if k < n_max:
            assert int(sel[u, k]) == -1, "index list written past k"
        # attention over the selected rows
        ref = O.attend(qg, K, V, idx_gpu)
        got = _np64(out[bi, h * G:(h + 1) * G])
        err = float(np.abs(ref - got).max())
        assert err <= tol, "attention output differs: max abs %g > %g (unit %d)" % (err, tol, u)
        report["out_max_abs_err"] = max(report.get("out_max_abs_err", 0.0), err)
        report["units_checked"] = report.get("units_checked", 0) + 1
    return out, sel


def check_append(sess: Session, k_new: torch.Tensor, v_new: torch.Tensor, units, report: dict):
    """bpc_append through the library: rows land at position n, the new code follows Algorithm 2, n advances."""
    s = sess.spec
    before = list(sess.lens)
    sess.ctx.append(k_new, v_new, sess.k_cache, sess.v_cache, sess.codes)
    torch.cuda.synchronize()
    assert sess.ctx.last_device_error() == 0
    sess.lens = [n + 1 for n in before]
    assert sess.ctx.get_seq_lens() == sess.lens
    for u in units:
        bi, h, n1 = sess.unit_views(u)
        n = n1 - 1
        assert torch.equal(sess.k_cache[bi, h, n], k_new[bi, h]) and torch.equal(sess.v_cache[bi, h, n], v_new[bi, h])
        check_encode(sess, [u], report, key_slice=(n, n + 1))


def check_yardsticks(sess: Session, q: torch.Tensor, units, report: dict, budget_ppm=None):
    """Quality yard-sticks through the library: bpc_exact_topk (per-head exact scores and top-k) and dense attention
    (the decode call with a budget of all keys), against the checker; then recall of the hash selection with respect to
    the exact top-k and the cosine similarity of sparse and dense outputs, computed on both sides."""
    s = sess.spec
    ppm = s.budget_ppm if budget_ppm is None else budget_ppm
    G = s.group
    scores, sel, cnt = sess.ctx.exact_topk(q, sess.k_cache, budget_ppm=ppm)
    dense = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=1000000)
    hsel = torch.full((sess.units, sess.w.n_max), -1, dtype=torch.int32, device="cuda")
    sparse = sess.ctx.decode_attn(q, sess.k_cache, sess.v_cache, sess.codes, budget_ppm=ppm, sel_idx=hsel)
    torch.cuda.synchronize()
    tol_out = 2e-3 if s.dtype == "bf16" else 1e-5
    rec_gpu, rec_ref, cos_all = [], [], []
    for u in units:
        bi, h, n = sess.unit_views(u)
        K = _np64(sess.k_cache[bi, h, :n]); V = _np64(sess.v_cache[bi, h, :n])
        qg = _np64(q[bi, h * G:(h + 1) * G])
        k = O.budget(n, ppm)
        hash_idx = hsel[u, :k].cpu().numpy().astype(np.int64)
        d_ref = O.dense_attend(qg, K, V)
        d_gpu = _np64(dense[bi, h * G:(h + 1) * G])
        assert np.abs(d_gpu - d_ref).max() <= tol_out * max(1.0, np.abs(d_ref).max()), "dense attention differs"
        s_gpu = _np64(sparse[bi, h * G:(h + 1) * G])
        for g in range(G):
            head = bi * s.n_q_heads + h * G + g
            sc64 = K @ qg[g]
            got_sc = _np64(scores[head, :n])
            assert np.abs(got_sc - sc64).max() <= 2e-5 * np.linalg.norm(qg[g]) * np.linalg.norm(K, axis=1).max(), "exact scores differ"
            assert int(cnt[head]) == k
            got = sel[head, :k].cpu().numpy().astype(np.int64)
            assert np.all(np.diff(got) > 0), "exact top-k list is not ascending"
            ref = O.exact_topk(qg[g], K, k)
            # keys on which the two selections disagree must sit at the k-th score within fp32 rounding
            kth = np.sort(sc64)[n - k]
            band = 4e-5 * np.linalg.norm(qg[g]) * np.linalg.norm(K, axis=1).max()
            diff = np.setxor1d(got, ref)
            assert np.all(np.abs(sc64[diff] - kth) <= band), "exact top-k differs outside the rounding band"
            rec_gpu.append(O.selection_recall(hash_idx, got)); rec_ref.append(O.selection_recall(hash_idx, ref))
            cos_all.append(O.cosine_similarity(s_gpu[g], d_gpu[g]))
            cref = O.cosine_similarity(O.attend(qg[g:g + 1], K, V, hash_idx)[0], d_ref[g])
            assert abs(cos_all[-1] - cref) <= 5e-3, "cosine of sparse vs dense output differs (%g vs %g)" % (cos_all[-1], cref)
        assert abs(np.mean(rec_gpu[-G:]) - np.mean(rec_ref[-G:])) <= 2.0 / max(k, 1)
    report["recall_vs_exact_topk"] = float(np.mean(rec_gpu))
    report["cosine_sparse_vs_dense"] = float(np.mean(cos_all))
