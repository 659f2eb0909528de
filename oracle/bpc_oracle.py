"""CPU checker for BinaryPC decode-time sparse attention (test infrastructure, not product code).

A plain, slow, fp64 restatement of what the hot path computes, written from the
paper's algorithms so that a reader can compare it with them by eye.  It shares
no code with the CUDA path and must never be imported by it: only the tests,
the smoke check and the benchmark's CPU-baseline leg may call it.

Notation follows the paper: N keys of dimension D, H-bit codes (here `b`),
projection P (b x D), codes h in {-1,+1}^b, residual R / r.

Readings taken where the paper is silent (each is listed in the design notes):
  * sign(0) = +1; a stored bit is 1 exactly when the component is +1.
  * bit j of a code (Algorithm iteration j+1) lives in 64-bit word j//64 at
    bit position j%64, least significant first.
  * the hash function is defined on P rounded to the cache precision (P_h).
  * the 7 magnitude planes carry weights 2^0..2^6, i.e. magnitudes in [0,127].
  * the projected query is quantised with a symmetric per-head abs-max scale,
    round-half-to-even, clamp at 127.
  * with grouped queries the per-head integer scores of a KV head are summed.
  * top-k ties go to the lowest index; the budget is ceil(n * ppm / 1e6).
  * softmax scale is 1/sqrt(D); the output is the plain softmax average.

Pins (tests/test_oracle_pins.py): Frobenius identity and orthogonality of
Algorithm 1, rank-1 closed form, least-squares optimality of v, greedy step
optimality and the orthogonal-P special case of Algorithm 2, Gram form vs
residual form, Hamming identity, bit-plane formula vs integer dot product
(exhaustive at 8 bits), brute-force sort for top-k, dense softmax at budget n,
scale invariance of query codes, storage arithmetic printed in the paper, safeguard set vs brute force and
its identity ||k - hP||^2 = ||k||^2 - 2 sum|t_i| + tr(P P^T) with the decision values t_i of Algorithm 2.
Parity unpinned: none of the functions below (the paper prints no numeric
worked example; every function has at least one mathematical pin).
"""
from __future__ import annotations

import math

import numpy as np

HAMMING = 0     # one magnitude plane, all magnitudes 1
WEIGHTED7 = 1   # sign + seven magnitude planes (Algorithm 3 as printed)


# --------------------------------------------------------------------------- rounding helpers
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32/fp64 values to the nearest bfloat16 (ties to even); returns float64 holding those values."""
    x32 = np.asarray(x, dtype=np.float32)
    bits = x32.view(np.uint32).astype(np.uint64)
    bias = np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))
    out = ((bits + bias) & np.uint64(0xFFFF0000)).astype(np.uint32)
    return out.view(np.float32).astype(np.float64)


def to_hash_precision(P: np.ndarray, dtype: str) -> np.ndarray:
    """P_h: the projection as the hash function uses it (bf16 caches -> bf16 values, fp32 caches -> fp32)."""
    p32 = np.asarray(P, dtype=np.float64).astype(np.float32)
    return round_bf16(p32) if dtype == "bf16" else p32.astype(np.float64)


def sign_pm1(t: np.ndarray) -> np.ndarray:
    """sign with sign(0) = +1, as float64 +-1."""
    return np.where(np.asarray(t) >= 0, 1.0, -1.0)


# --------------------------------------------------------------------------- Algorithm 1
def fit(K: np.ndarray, v_star: np.ndarray, power_iters: int = 0):
    """Algorithm 1: greedy binary principal components.

    K [N, D], v_star [b, D] (the Gaussian draws, passed in).  Returns
    P [b, D], H [N, b] in {-1,+1}, and the residual Frobenius norms after 0..b iterations.

    power_iters = n > 0 takes the binary component from the power iteration the section "Binary Principal
    Components Finding" starts from, u = sign((R R^T)^n R v*^T); n = 0 is Algorithm 1 as printed, u = sign(R v*^T).
    The vector is rescaled between multiplications (a positive factor: the signs are those of the formula).
    """
    R = np.array(K, dtype=np.float64)
    N = R.shape[0]
    b = v_star.shape[0]
    P = np.zeros((b, R.shape[1]))
    H = np.zeros((N, b))
    trace = [np.linalg.norm(R)]
    for i in range(b):
        w = R @ np.asarray(v_star[i], dtype=np.float64)              # R v*^T
        for _ in range(power_iters):                                 # (R R^T)^n applied one factor at a time
            nw = np.linalg.norm(w)
            if nw > 0.0:
                w = w / nw
            w = R @ (R.T @ w)
        u = sign_pm1(w)                                              # binary component of this iteration
        v = (u @ R) / N                                              # its least-squares row of P
        R = R - np.outer(u, v)                                       # what the component explains is removed
        H[:, i] = u
        P[i, :] = v
        trace.append(np.linalg.norm(R))
    return P, H, np.array(trace)


# --------------------------------------------------------------------------- Algorithm 2
def encode(K: np.ndarray, P_h: np.ndarray, residual_correction: bool = True):
    """Algorithm 2 for every row of K [n, D] with projection P_h [b, D].

    Returns bits [n, b] (uint8, 1 <=> +1) and the final residual norms ||k - h P||_2 (Eq. 8).
    With residual_correction False the residual is never updated (plain sign(k P^T)).
    """
    r = np.array(K, dtype=np.float64)
    P_h = np.asarray(P_h, dtype=np.float64)
    b = P_h.shape[0]
    bits = np.zeros((r.shape[0], b), dtype=np.uint8)
    for i in range(b):
        v = P_h[i]
        u = sign_pm1(r @ v)
        if residual_correction:
            r = r - u[:, None] * v[None, :]
        bits[:, i] = (u > 0)
    if not residual_correction:
        h = 2.0 * bits - 1.0
        r = np.array(K, dtype=np.float64) - h @ P_h
    return bits, np.linalg.norm(r, axis=1)


def pack_bits(bits: np.ndarray) -> np.ndarray:
    """bits [n, b] -> uint64 words [n, b/64]; bit j -> word j//64, position j%64 (LSB first)."""
    n, b = bits.shape
    assert b % 64 == 0
    out = np.zeros((n, b // 64), dtype=np.uint64)
    for j in range(b):
        out[:, j // 64] |= bits[:, j].astype(np.uint64) << np.uint64(j % 64)
    return out


def unpack_bits(words: np.ndarray, b: int) -> np.ndarray:
    words = np.asarray(words, dtype=np.uint64)
    out = np.zeros((words.shape[0], b), dtype=np.uint8)
    for j in range(b):
        out[:, j] = ((words[:, j // 64] >> np.uint64(j % 64)) & np.uint64(1)).astype(np.uint8)
    return out


def codes_bytes(n_keys: int, b: int) -> int:
    """Storage of the packed codes: b/8 bytes per key and KV head (Appendix: one int64 per key at 64 bits)."""
    return n_keys * b // 8


# --------------------------------------------------------------------------- query hash (Retrieval Phase)
def query_hash(q_group: np.ndarray, P_h: np.ndarray, mode: int):
    """Projected, quantised queries of one KV head.

    q_group [G, D].  Returns p [G, b] (fp64 projection q P^T), s [G, b] in {-1,+1},
    a [G, b] integer magnitudes (all 1 in HAMMING mode; 0..127 in WEIGHTED7 mode).
    """
    q = np.asarray(q_group, dtype=np.float64)
    p = q @ np.asarray(P_h, dtype=np.float64).T
    s = sign_pm1(p)
    if mode == HAMMING:
        a = np.ones_like(p, dtype=np.int64)
    else:
        a = np.zeros_like(p, dtype=np.int64)
        for g in range(p.shape[0]):
            pmax = np.max(np.abs(p[g]))
            if pmax > 0:
                a[g] = np.minimum(127, np.rint((127.0 * np.abs(p[g])) / pmax)).astype(np.int64)
    return p, s, a


def collapsed_weights(s: np.ndarray, a: np.ndarray) -> np.ndarray:
    """A = sum_g s_g * a_g (integer vector of length b): the group score is <A, h>."""
    return np.sum(s.astype(np.int64) * a, axis=0)


# --------------------------------------------------------------------------- hash score
def hash_scores(bits: np.ndarray, s: np.ndarray, a: np.ndarray) -> np.ndarray:
    """c = (quantised q P^T) h^T summed over the query heads of the group, for every key.

    bits [n, b] in {0,1}; s, a [G, b].  Exact integers (int64) [n].
    """
    h = 2 * bits.astype(np.int64) - 1
    w = s.astype(np.int64) * a.astype(np.int64)          # [G, b]
    return (h @ w.T).sum(axis=1)


def hash_score_alg3(h_bits: np.ndarray, s_neg_bits: np.ndarray, mag_planes: np.ndarray) -> int:
    """Algorithm 3 for one key and one query head, evaluated on bit vectors.

    h_bits [b] (1 <=> h=+1), s_neg_bits [b] (1 <=> query sign negative), mag_planes [7, b] in {0,1}
    with plane j weighted 2^j.  w = h XOR s marks the positions whose product h*s is +1.
    """
    w = np.bitwise_xor(h_bits.astype(np.uint8), s_neg_bits.astype(np.uint8))
    c = 0
    for j in range(mag_planes.shape[0]):
        m = int(np.count_nonzero(w & mag_planes[j])) - int(np.count_nonzero((1 - w) & mag_planes[j]))
        c += m << j
    return c


def magnitude_planes(a_row: np.ndarray, planes: int = 7) -> np.ndarray:
    return np.array([(a_row >> j) & 1 for j in range(planes)], dtype=np.uint8)


def hamming_distance(words_a: np.ndarray, words_b: np.ndarray) -> int:
    x = np.bitwise_xor(np.asarray(words_a, dtype=np.uint64), np.asarray(words_b, dtype=np.uint64))
    return int(sum(bin(int(v)).count("1") for v in np.atleast_1d(x)))


# --------------------------------------------------------------------------- selection
def budget(n: int, ppm: int, count: int = 0) -> int:
    """Number of keys kept: a fixed count if given, else ceil(n * ppm / 1e6); never more than n."""
    k = count if count > 0 else -(-n * ppm // 1000000)
    return max(0, min(n, k))


def topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k highest scores, ties to the lowest index, returned in ascending index order."""
    scores = np.asarray(scores)
    order = np.lexsort((np.arange(scores.shape[0]), -scores.astype(np.int64)))
    return np.sort(order[:k]).astype(np.int64)


# --------------------------------------------------------------------------- attention over the selected rows
def attend(q_group: np.ndarray, K: np.ndarray, V: np.ndarray, idx: np.ndarray, sm_scale: float = 0.0) -> np.ndarray:
    """softmax(sm_scale * q K_S^T) V_S for each query head of the group; S = idx.  Returns [G, D] fp64."""
    q = np.asarray(q_group, dtype=np.float64)
    Ks = np.asarray(K, dtype=np.float64)[idx]
    Vs = np.asarray(V, dtype=np.float64)[idx]
    if sm_scale == 0.0:
        sm_scale = 1.0 / math.sqrt(q.shape[1])
    logits = sm_scale * (q @ Ks.T)
    logits = logits - logits.max(axis=1, keepdims=True)
    w = np.exp(logits)
    w = w / w.sum(axis=1, keepdims=True)
    return w @ Vs


# --------------------------------------------------------------------------- quality yard-sticks
def exact_topk(q_head: np.ndarray, K: np.ndarray, k: int) -> np.ndarray:
    """The TOPK (Oracle) baseline of the appendix "Baseline Methods": the k keys with the largest exact attention
    scores q . k_i for ONE query head (full precision), ties to the lowest index, returned in ascending index order."""
    scores = np.asarray(K, dtype=np.float64) @ np.asarray(q_head, dtype=np.float64)
    k = max(0, min(int(k), scores.shape[0]))
    order = np.lexsort((np.arange(scores.shape[0]), -scores))
    return np.sort(order[:k]).astype(np.int64)


def dense_attend(q_group: np.ndarray, K: np.ndarray, V: np.ndarray, sm_scale: float = 0.0) -> np.ndarray:
    """Full softmax attention over every cached key (the reference the sparse output is compared with)."""
    return attend(q_group, K, V, np.arange(np.asarray(K).shape[0]), sm_scale)


def selection_recall(selected: np.ndarray, reference: np.ndarray) -> float:
    """Fraction of the reference set that the selection contains."""
    reference = np.asarray(reference)
    if reference.size == 0:
        return 1.0
    return float(np.isin(reference, np.asarray(selected)).mean())


def cosine_similarity(a: np.ndarray, b: np.ndarray) -> float:
    """cos(a, b) of two vectors (appendix table "cosine similarity between sparse and full attention outputs")."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = np.linalg.norm(a) * np.linalg.norm(b)
    return float(a @ b / den) if den > 0.0 else 0.0


# --------------------------------------------------------------------------- Error-Aware Safeguard (Eqs. 8-9)
def eas_set(errors: np.ndarray, m: int) -> np.ndarray:
    """Hard-to-hash set S_err: indices of the m largest reconstruction errors ||k - h P||_2 (Eq. 8), ties to the
    lowest index, returned in ascending index order.  It is built once, at prefill."""
    errors = np.asarray(errors, dtype=np.float64)
    order = np.lexsort((np.arange(errors.shape[0]), -errors))
    return np.sort(order[:max(0, min(m, errors.shape[0]))]).astype(np.int64)


def eas_union(hash_idx: np.ndarray, s_err: np.ndarray) -> np.ndarray:
    """S_attn = S_hash united with S_err (Eq. 9), ascending."""
    return np.union1d(np.asarray(hash_idx, dtype=np.int64), np.asarray(s_err, dtype=np.int64))


# --------------------------------------------------------------------------- one decode step of one unit
def decode_unit(q_group, K, V, bits, P_h, ppm, count=0, mode=HAMMING, sm_scale=0.0, s_err=None):
    """Query hash -> scores over all cached keys -> top-k -> attention.  K, V, bits hold the n cached rows.

    With an error-aware safeguard set s_err (ascending indices), the budget k is split: the first min(|s_err|, k)
    safeguard keys are always attended and the hash search fills the remaining k - min(|s_err|, k) places
    (it competes over all keys, so a key may be chosen twice; the union removes it).  When the set is larger than
    the budget (the paper sizes it at a tenth of the budget, so this is a degenerate case it never meets) "the first"
    means the lowest indices: the set is static and kept in index order, its members are not ranked again by error.
    Returns dict(out [G, D], idx [<= k] (attended keys, ascending), hash_idx, scores [n], s, a).
    """
    _, s, a = query_hash(q_group, P_h, mode)
    sc = hash_scores(bits, s, a)
    k = budget(bits.shape[0], ppm, count)
    if s_err is None:
        hash_idx = topk(sc, k)
        idx = hash_idx
    else:
        me = min(len(s_err), k)
        hash_idx = topk(sc, k - me)
        idx = eas_union(hash_idx, np.asarray(s_err)[:me])
    out = attend(q_group, K, V, idx, sm_scale)
    return dict(out=out, idx=idx, hash_idx=hash_idx, scores=sc, s=s, a=a)


def ambiguity_threshold_query(q_row: np.ndarray, P_h: np.ndarray, rel: float = 1e-6) -> np.ndarray:
    """Per-bit magnitude below which a query sign bit may legitimately differ: rel * ||q|| * ||P_j||."""
    return rel * np.linalg.norm(q_row) * np.linalg.norm(P_h, axis=1)


def replay_encode_with_adoption(K: np.ndarray, P_h: np.ndarray, other_bits: np.ndarray, rel: float = 1e-6):
    """Replay Algorithm 2 in fp64 for keys K [n, D] against another implementation's bits [n, b].

    At iteration i the decision value is t = r . P_i.  Where the other side's bit differs while |t| is at
    least tau_i = rel * (||k|| ||P_i|| + sum_{j<i} |P_j . P_i|) it is a hard mismatch; below tau_i the bit
    is ambiguous.  Either way the other side's bit is adopted and the replay continues from it, so one
    early ambiguous decision does not condemn the rest of the code.
    Returns (hard [n, b] bool, ambiguous [n, b] bool).
    """
    P_h = np.asarray(P_h, dtype=np.float64)
    r = np.array(K, dtype=np.float64)
    knorm = np.linalg.norm(r, axis=1)
    pn = np.linalg.norm(P_h, axis=1)
    b = P_h.shape[0]
    hard = np.zeros((r.shape[0], b), dtype=bool)
    amb = np.zeros((r.shape[0], b), dtype=bool)
    for i in range(b):
        t = r @ P_h[i]
        mine = (t >= 0)
        theirs = other_bits[:, i].astype(bool)
        tau = rel * (knorm * pn[i] + float(np.sum(np.abs(P_h[:i] @ P_h[i]))))
        diff = mine != theirs
        hard[:, i] = diff & (np.abs(t) >= tau)
        amb[:, i] = diff & (np.abs(t) < tau)
        u = np.where(theirs, 1.0, -1.0)
        r = r - u[:, None] * P_h[i][None, :]
    return hard, amb
