"""Pins for the CPU oracle: hand-worked fixtures, closed forms, invariants, library routines
and brute force. None of these tests touches the CUDA library."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import ec_oracle as orc
from paper_2407_18121_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _bf16(x):
    return wl.to_bf16_bits(np.asarray(x, np.float32))


def _rand_bits(rng, shape, sigma=1.0):
    return _bf16(rng.standard_normal(shape).astype(np.float32) * sigma)


# ------------------------------------------------------------------ importance (Eq. 1)

def test_importance_hand_example():
    rows = _rows("importance_pow2.txt")
    q = _bf16(np.ones((1, 3, 1)))
    k = _bf16(np.array([0.0, 1.0, 2.0]).reshape(1, 3, 1))
    scores, lse = orc.importance(q, k, math.log(2.0))
    want = np.array([float(Fraction(int(a), int(b))) for a, b, _ in rows])
    want_lse = np.array([math.log(float(c)) for _, _, c in rows])
    np.testing.assert_allclose(scores[0], want, rtol=1e-14)
    np.testing.assert_allclose(lse[0], want_lse, rtol=0, atol=1e-14)


def test_importance_zero_queries_is_harmonic():
    # uniform attention: I_n = sum_{m>=n} 1/(m+1) = H_T - H_n
    T, D = 37, 8
    rng = np.random.default_rng(0)
    q = _bf16(np.zeros((2, T, D)))
    k = _rand_bits(rng, (2, T, D))
    scores, lse = orc.importance(q, k, 0.7)
    want = np.array([sum(1.0 / (m + 1) for m in range(n, T)) for n in range(T)])
    np.testing.assert_allclose(scores[0], want, rtol=1e-13)
    np.testing.assert_allclose(scores[1], want, rtol=1e-13)
    np.testing.assert_allclose(lse[0], np.log(np.arange(1, T + 1)), atol=1e-13)


@pytest.mark.parametrize("T,D,scale", [(1, 4, 1.0), (2, 4, 0.3), (16, 8, 1.0), (45, 16, 0.25)])
def test_importance_matches_library_softmax(T, D, scale):
    rng = np.random.default_rng(T * 100 + D)
    qb, kb = _rand_bits(rng, (3, T, D)), _rand_bits(rng, (3, T, D))
    scores, lse = orc.importance(qb, kb, scale)
    q = torch.from_numpy(wl.bf16_bits_to_f64(qb))
    k = torch.from_numpy(wl.bf16_bits_to_f64(kb))
    logits = scale * q @ k.transpose(-1, -2)
    mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
    logits = logits.masked_fill(~mask, float("-inf"))
    A = torch.softmax(logits, dim=-1)
    np.testing.assert_allclose(scores, A.sum(dim=-2).numpy(), rtol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-12, atol=1e-12)


def test_importance_operands_not_transposed():
    # asymmetric case: only the q.k order that puts QUERIES on rows gives this answer
    T, D = 5, 3
    rng = np.random.default_rng(5)
    qb, kb = _rand_bits(rng, (1, T, D), 2.0), _rand_bits(rng, (1, T, D), 2.0)
    s_qk, _ = orc.importance(qb, kb, 1.0)
    s_kq, _ = orc.importance(kb, qb, 1.0)
    assert np.abs(s_qk - s_kq).max() > 1e-3
    q, k = wl.bf16_bits_to_f64(qb)[0], wl.bf16_bits_to_f64(kb)[0]
    I = np.zeros(T)
    for m in range(T):
        w = np.array([math.exp(float(q[m] @ k[n])) for n in range(m + 1)])
        I[: m + 1] += w / w.sum()
    np.testing.assert_allclose(s_qk[0], I, rtol=1e-12)


def test_importance_invariants():
    T, D = 64, 16
    rng = np.random.default_rng(7)
    qb, kb = _rand_bits(rng, (4, T, D)), _rand_bits(rng, (4, T, D))
    scores, _ = orc.importance(qb, kb, 0.5)
    np.testing.assert_allclose(scores.sum(-1), T, rtol=1e-12)   # rows of A sum to one
    assert (scores[:, 0] >= 1.0).all()                           # A[0][0] = 1
    assert (scores[:, -1] <= 1.0).all() and (scores > 0).all()


def test_layer_mean():
    rng = np.random.default_rng(1)
    s = rng.random((3, 5, 11))
    np.testing.assert_allclose(orc.layer_mean(s), s.mean(axis=1), rtol=1e-14)


# ------------------------------------------------------------------ keep count / selection

def test_keep_counts_of_the_five_configurations():
    got = []
    for name in wl.CONFIG_ORDER:
        w = wl.WORKLOADS[name]
        got.append([orc.keep_count(w.prompt_len, r) for r in w.keep_ratios])
    assert got == [[128], [320], [256], [205, 512, 1024, 1536], [820]]
    assert orc.keep_count(100, 1.0) == 100 and orc.keep_count(100, 0.0) == 1


def _brute_select(s, C, protect):
    s = np.array(s, np.float64)
    T = len(s)
    if protect:
        s[0] = np.inf
        if C >= 2:
            s[-1] = np.inf
    order = sorted(range(T), key=lambda i: (-s[i], i))
    return np.array(sorted(order[:C]), np.int32)


@pytest.mark.parametrize("protect", [False, True])
def test_select_brute_force_with_ties(protect):
    rng = np.random.default_rng(3)
    for T, C in [(1, 1), (2, 1), (2, 2), (9, 1), (9, 4), (33, 33), (40, 17)]:
        s = rng.integers(0, 6, size=(5, T)).astype(np.float64)   # many exact ties
        got = orc.select(s, C, protect)
        for u in range(5):
            np.testing.assert_array_equal(got[u], _brute_select(s[u], C, protect))


def test_select_known_top_set_and_order():
    s = np.array([[0.1, 5.0, 0.2, 4.0, 0.3, 3.0, 0.0]])
    np.testing.assert_array_equal(orc.select(s, 3, False)[0], [1, 3, 5])
    np.testing.assert_array_equal(orc.select(s, 3, True)[0], [0, 1, 6])
    np.testing.assert_array_equal(orc.select(s, 7, False)[0], np.arange(7))
    # lower position wins a tie
    t = np.array([[1.0, 2.0, 2.0, 2.0]])
    np.testing.assert_array_equal(orc.select(t, 2, False)[0], [1, 2])


def test_select_threshold_property():
    rng = np.random.default_rng(11)
    s = rng.random((6, 200))
    a = orc.select(s, 50, False)
    for u in range(6):
        assert (np.diff(a[u]) > 0).all() and len(a[u]) == 50
        rest = np.setdiff1d(np.arange(200), a[u])
        assert s[u, a[u]].min() >= s[u, rest].max()


# ------------------------------------------------------------------ buckets (Eq. 2), merge (Eq. 3)

def test_bucket_merge_hand_example():
    rows = _rows("bucket_merge_example.txt")
    T, D = 7, 2
    X = np.array([[t, 10 - 2 * t] for t in range(T)], np.float32).reshape(1, T, D)
    anchors = np.array([[0, 3, 4]], np.int32)
    lo, hi = orc.buckets(anchors, T)
    assert lo[0].tolist() == [int(r[0]) for r in rows]
    assert hi[0].tolist() == [int(r[1]) for r in rows]
    m = orc.merge(_bf16(X), lo, hi)
    want = np.array([[float(r[2]), float(r[3])] for r in rows])
    np.testing.assert_allclose(m[0], want, rtol=1e-15)


def test_buckets_are_nearest_anchor_ties_to_earlier():
    rng = np.random.default_rng(2)
    for T, C in [(1, 1), (5, 1), (8, 8), (30, 7), (64, 20), (65, 2)]:
        a = np.sort(rng.choice(T, size=C, replace=False)).astype(np.int32)[None]
        lo, hi = orc.buckets(a, T)
        owner = np.full(T, -1)
        for k in range(C):
            assert lo[0, k] <= a[0, k] <= hi[0, k]
            assert (owner[lo[0, k]: hi[0, k] + 1] == -1).all()
            owner[lo[0, k]: hi[0, k] + 1] = k
        assert (owner >= 0).all()
        for t in range(T):
            d = np.abs(a[0].astype(np.int64) - t)
            assert owner[t] == int(np.argmin(d))     # argmin returns the first = earlier anchor


def test_merge_properties():
    rng = np.random.default_rng(4)
    U, T, D, C = 3, 50, 8, 9
    Xb = _rand_bits(rng, (U, T, D))
    X = wl.bf16_bits_to_f64(Xb)
    anchors = np.stack([np.sort(rng.choice(T, C, replace=False)) for _ in range(U)]).astype(np.int32)
    lo, hi = orc.buckets(anchors, T)
    m = orc.merge(Xb, lo, hi)
    size = (hi - lo + 1).astype(np.float64)
    np.testing.assert_allclose((m * size[..., None]).sum(1), X.sum(1), rtol=1e-12, atol=1e-12)
    # explicit per-bucket numpy mean
    for u in range(U):
        for k in range(C):
            np.testing.assert_allclose(m[u, k], X[u, lo[u, k]: hi[u, k] + 1].mean(0), rtol=1e-13, atol=1e-15)
    # one anchor: global mean; all anchors: identity, bit for bit after rounding back
    one = np.array([[17]] * U, np.int32)
    l1, h1 = orc.buckets(one, T)
    np.testing.assert_allclose(orc.merge(Xb, l1, h1)[:, 0], X.mean(1), rtol=1e-13)
    full = np.tile(np.arange(T, dtype=np.int32), (U, 1))
    lf, hf = orc.buckets(full, T)
    np.testing.assert_array_equal(orc.round_bf16(orc.merge(Xb, lf, hf)), Xb)
    # constant rows stay constant
    const = _bf16(np.full((1, 20, 4), 1.5))
    lc, hc = orc.buckets(np.array([[3, 9, 15]], np.int32), 20)
    assert (orc.merge(const, lc, hc) == 1.5).all()


def test_round_bf16_is_round_to_nearest_even():
    # 1 + 2^-8 is the midpoint between bf16 neighbours 1 and 1 + 2^-7: tie goes to even (1.0)
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -30, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0, 1e-3])
    got = wl.bf16_bits_to_f64(orc.round_bf16(x))
    assert got[0] == 1.0 and got[1] == 1.0 + 2.0 ** -7 and got[2] == 1.0 + 2.0 ** -6 and got[3] == -2.5
    assert got[4] == 0.0 and abs(got[5] - 1e-3) <= 1e-3 * 2.0 ** -8
    # agrees with torch's float32 -> bfloat16 on float32-representable values
    rng = np.random.default_rng(0)
    f = rng.standard_normal(4096).astype(np.float32)
    tb = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(orc.round_bf16(f.astype(np.float64)), tb)
    np.testing.assert_array_equal(wl.to_bf16_bits(f), tb)
    np.testing.assert_array_equal(orc.widen_bf16(tb), torch.from_numpy(tb.view(np.int16)).view(torch.bfloat16).double().numpy())


# ------------------------------------------------------------------ decode attention + eviction

def test_decode_hand_example():
    want = float(_rows("decode_pow2.txt")[0][0])
    K0 = np.array([[0.0], [1.0]]).reshape(1, 2, 1)
    V0 = np.array([[1.0], [2.0]]).reshape(1, 2, 1)
    qd = orc.DecodeQueue(K0, V0, cap=4)
    out, pos, ident = qd.step(_bf16([[1.0]]), _bf16([[2.0]]), _bf16([[4.0]]), math.log(2.0),
                              policy=orc.POLICY_FIXED, budget=8, offset=1)
    assert abs(out[0, 0] - want) < 1e-14 and pos == -1 and ident == -1 and qd.len == 3


def test_decode_matches_library_softmax_and_special_cases():
    rng = np.random.default_rng(9)
    U, L, D = 4, 23, 16
    K0 = wl.bf16_bits_to_f64(_rand_bits(rng, (U, L, D)))
    V0 = wl.bf16_bits_to_f64(_rand_bits(rng, (U, L, D)))
    qb, kb, vb = _rand_bits(rng, (U, D)), _rand_bits(rng, (U, D)), _rand_bits(rng, (U, D))
    qd = orc.DecodeQueue(K0, V0, cap=L + 1)
    out, _, _ = qd.step(qb, kb, vb, 0.25, policy=orc.POLICY_FIXED, budget=L + 1, offset=3)
    Kall = torch.from_numpy(np.concatenate([K0, wl.bf16_bits_to_f64(kb)[:, None]], 1))
    Vall = torch.from_numpy(np.concatenate([V0, wl.bf16_bits_to_f64(vb)[:, None]], 1))
    q = torch.from_numpy(wl.bf16_bits_to_f64(qb))
    p = torch.softmax(0.25 * torch.einsum("ud,uld->ul", q, Kall), dim=-1)
    want = torch.einsum("ul,uld->ud", p, Vall).numpy()
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-14)
    # convex combination
    assert (out <= Vall.numpy().max(1) + 1e-12).all() and (out >= Vall.numpy().min(1) - 1e-12).all()
    # q = 0 -> plain mean of all value rows (cache and new)
    qd0 = orc.DecodeQueue(K0, V0, cap=L + 1)
    out0, _, _ = qd0.step(_bf16(np.zeros((U, D))), kb, vb, 0.25, policy=0, budget=L + 1, offset=3)
    np.testing.assert_allclose(out0, Vall.numpy().mean(1), rtol=1e-13, atol=1e-15)
    # permuting cached rows leaves the output unchanged
    perm = rng.permutation(L)
    qdp = orc.DecodeQueue(K0[:, perm], V0[:, perm], cap=L + 1)
    outp, _, _ = qdp.step(qb, kb, vb, 0.25, policy=0, budget=L + 1, offset=3)
    np.testing.assert_allclose(outp, out, rtol=1e-12, atol=1e-14)


def test_fixed_point_queue_hand_example():
    rows = _rows("fixed_point_queue.txt")
    rng = np.random.default_rng(0)
    K0 = rng.standard_normal((2, 5, 4))
    qd = orc.DecodeQueue(K0, K0.copy(), cap=6)
    for r in rows:
        kb = _rand_bits(rng, (2, 4))
        _, pos, ident = qd.step(kb, kb, kb, 1.0, policy=orc.POLICY_FIXED, budget=5, offset=2)
        assert pos == int(r[1]) and ident == int(r[2])
        assert qd.identities().tolist() == [int(x) for x in r[3:]]


def test_fixed_point_retained_set_and_contents():
    rng = np.random.default_rng(12)
    C, d, D, steps = 12, 4, 4, 19
    K0 = wl.bf16_bits_to_f64(_rand_bits(rng, (1, C, D)))
    qd = orc.DecodeQueue(K0, K0.copy(), cap=C + 1)
    newk = []
    for s in range(steps):
        kb = _rand_bits(rng, (1, D))
        newk.append(wl.bf16_bits_to_f64(kb)[0])
        _, pos, ident = qd.step(kb, kb, kb, 1.0, policy=0, budget=C, offset=d)
        assert qd.len == C and pos == C - d                      # fixed truncation location
        ids = qd.identities()
        recent = list(range(C + s - d + 1, C + s + 1))
        assert ids.tolist() == list(range(C - d)) + recent       # first C-d rows + d newest
        assert ident == (C - d + s)                              # rows leave in arrival order
        for j, i in enumerate(ids):                              # rows moved with their identities
            src = K0[0, i] if i < C else newk[i - C]
            np.testing.assert_array_equal(qd.K[0, j], src)


def test_below_budget_nothing_is_evicted():
    rng = np.random.default_rng(13)
    K0 = rng.standard_normal((1, 3, 4))
    qd = orc.DecodeQueue(K0, K0.copy(), cap=8)
    for s in range(4):
        kb = _rand_bits(rng, (1, 4))
        _, pos, _ = qd.step(kb, kb, kb, 1.0, policy=0, budget=6, offset=2)
        assert pos == (-1 if s < 3 else 4)
    assert qd.len == 6


def _golden_rows(name):
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    return [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]


def test_ratio_policy_hand_worked_traces():
    """Two traces worked by hand from Algorithm 1's del_num line (tests/golden/retention_ratio_queue.txt):
    which steps grow, which evict, which identity leaves and the queue after every step. They fix the
    conventions a shared mistake could hide: the new token is counted in n, and seq_len is the length
    after the append."""
    rows = _golden_rows("retention_ratio_queue.txt")
    cases = {}
    for r in rows:
        cases.setdefault((r[0], int(r[1]), float(r[2]), int(r[3])), []).append(
            (int(r[4]), int(r[5]), int(r[6]), [int(x) for x in r[7:]]))
    assert len(cases) == 2
    rng = np.random.default_rng(15)
    for (_, T, ratio, offset), steps in cases.items():
        C = orc.keep_count(T, ratio)
        assert C == len(steps[0][3]) - (1 if steps[0][1] < 0 else 0)
        K0 = rng.standard_normal((2, C, 4))
        qd = orc.DecodeQueue(K0, K0.copy(), cap=C + len(steps) + 1, n_seen=T)
        for s, pos_want, id_want, ids_want in steps:
            kb = _rand_bits(rng, (2, 4))
            _, pos, ident = qd.step(kb, kb, kb, 1.0, policy=orc.POLICY_RATIO, offset=offset, ratio=ratio)
            assert (pos, ident) == (pos_want, id_want), (T, ratio, s)
            assert qd.identities().tolist() == ids_want, (T, ratio, s)
            assert qd.n_seen == T + s + 1


def test_keep_count_hand_worked_cases():
    """Cases where the readings of N_I = gamma*T differ (tests/golden/keep_count_cases.txt): Algorithm 1's
    int(T - T*gamma) removed rows is the one taken."""
    rows = _golden_rows("keep_count_cases.txt")
    assert len(rows) >= 6
    for T, g, kept, other in rows:
        assert orc.keep_count(int(T), float(g)) == int(kept) != int(other)


def test_ratio_policy_follows_algorithm_1_count():
    # direct simulation of del_num = int(seq_len - n * ratio): one row leaves whenever it reaches 1
    rng = np.random.default_rng(14)
    T, ratio, d = 40, 0.3, 5
    C = orc.keep_count(T, ratio)
    K0 = rng.standard_normal((1, C, 4))
    qd = orc.DecodeQueue(K0, K0.copy(), cap=C + 40, n_seen=T)
    length = C
    for s in range(30):
        n_tot = T + s + 1
        kb = _rand_bits(rng, (1, 4))
        _, pos, _ = qd.step(kb, kb, kb, 1.0, policy=orc.POLICY_RATIO, offset=d, ratio=ratio)
        length += 1
        if int(length - n_tot * ratio) >= 1:
            assert pos == length - 1 - d
            length -= 1
        else:
            assert pos == -1
        assert qd.len == length
        assert length <= n_tot * ratio + 1


# ------------------------------------------------------------------ ablation variants

def test_group_mean_and_gather_reduce_to_numpy():
    rng = np.random.default_rng(31)
    s = rng.random((12, 17))
    np.testing.assert_allclose(orc.group_mean(s, 4), s.reshape(3, 4, 17).mean(1), rtol=1e-14)
    np.testing.assert_allclose(orc.group_mean(s, 1), s, rtol=0)
    np.testing.assert_allclose(orc.group_mean(s, 12)[0], s.mean(0), rtol=1e-14)
    np.testing.assert_allclose(orc.group_mean(s, 4), orc.layer_mean(s.reshape(3, 4, 17)), rtol=1e-15)
    Xb = _rand_bits(rng, (2, 9, 4))
    a = np.array([[0, 3, 8], [1, 2, 7]], np.int32)
    got = orc.gather(Xb, a)
    X = wl.bf16_bits_to_f64(Xb)
    for u in range(2):
        np.testing.assert_array_equal(got[u], X[u, a[u]])


def test_importance_prefix_matches_library_softmax_and_reduces_to_plain():
    rng = np.random.default_rng(41)
    for Tq, P, D in [(1, 0, 4), (5, 3, 4), (17, 40, 8), (30, 1, 8)]:
        qb, kb = _rand_bits(rng, (2, Tq, D)), _rand_bits(rng, (2, P + Tq, D))
        scores, lse = orc.importance_prefix(qb, kb, 0.4)
        q = torch.from_numpy(wl.bf16_bits_to_f64(qb))
        k = torch.from_numpy(wl.bf16_bits_to_f64(kb))
        logits = 0.4 * q @ k.transpose(-1, -2)                           # [2, Tq, P+Tq]
        m_idx = torch.arange(Tq)[:, None]
        n_idx = torch.arange(P + Tq)[None, :]
        logits = logits.masked_fill(n_idx > m_idx + P, float("-inf"))     # query m sees keys n <= m + P
        A = torch.softmax(logits, dim=-1)
        np.testing.assert_allclose(scores, A.sum(dim=-2).numpy(), rtol=1e-12)
        np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(scores.sum(-1), Tq, rtol=1e-12)       # one unit of mass per query
        if P == 0:
            s0, l0 = orc.importance(qb, kb, 0.4)
            np.testing.assert_array_equal(scores, s0)
            np.testing.assert_array_equal(lse, l0)


# ------------------------------------------------------------------ other importance statistics (Sec. 3.2)

def _attention_rows(qb, kb, scale):
    """A [U, Tq, P+Tq] from library routines (fp64 matmul + softmax), zero past the causal limit."""
    q = torch.from_numpy(wl.bf16_bits_to_f64(qb))
    k = torch.from_numpy(wl.bf16_bits_to_f64(kb))
    Tq, Tk = q.shape[-2], k.shape[-2]
    logits = scale * q @ k.transpose(-1, -2)
    m_idx, n_idx = torch.arange(Tq)[:, None], torch.arange(Tk)[None, :]
    logits = logits.masked_fill(n_idx > m_idx + (Tk - Tq), float("-inf"))
    return torch.softmax(logits, dim=-1)


def test_statistics_hand_example():
    # two tokens, one dimension, q = 1, k = (0, 1), scale = ln 2: A = [[1, 0], [1/3, 2/3]]
    q = _bf16(np.ones((1, 2, 1)))
    k = _bf16(np.array([0.0, 1.0]).reshape(1, 2, 1))
    sc = math.log(2.0)
    np.testing.assert_allclose(orc.importance_statistic(q, k, sc, orc.STAT_SUM)[0], [4 / 3, 2 / 3], rtol=1e-14)
    np.testing.assert_allclose(orc.importance_statistic(q, k, sc, orc.STAT_MEAN)[0], [2 / 3, 2 / 3], rtol=1e-14)
    np.testing.assert_allclose(orc.importance_statistic(q, k, sc, orc.STAT_MAX)[0], [1.0, 2 / 3], rtol=1e-14)
    # beta = 1/4: E = (3/4, 0) after the first query, then (1/4)(3/4) + (3/4)(1/3) = 7/16 and (3/4)(2/3) = 1/2
    np.testing.assert_allclose(orc.importance_statistic(q, k, sc, orc.STAT_MOVING_AVERAGE, 0.25)[0], [7 / 16, 1 / 2],
                               rtol=1e-14)


def test_statistics_uniform_attention_closed_forms():
    # zero queries: A[m][n] = 1/(m + P + 1) for n <= m + P
    Tq, P, D, beta = 9, 4, 4, Fraction(2, 3)
    rng = np.random.default_rng(5)
    q = _bf16(np.zeros((1, Tq, D)))
    k = _rand_bits(rng, (1, P + Tq, D))
    first = [max(0, n - P) for n in range(P + Tq)]                      # first query that sees key n
    mean = [sum(Fraction(1, m + P + 1) for m in range(first[n], Tq)) / (Tq - first[n]) for n in range(P + Tq)]
    mx = [Fraction(1, first[n] + P + 1) for n in range(P + Tq)]         # the earliest visible row is the largest
    ema = [sum((1 - beta) * beta ** (Tq - 1 - m) * Fraction(1, m + P + 1) for m in range(first[n], Tq))
           for n in range(P + Tq)]
    for stat, want, b in [(orc.STAT_MEAN, mean, 0.0), (orc.STAT_MAX, mx, 0.0), (orc.STAT_MOVING_AVERAGE, ema, float(beta))]:
        got = orc.importance_statistic(q, k, 0.9, stat, b)[0]
        np.testing.assert_allclose(got, [float(w) for w in want], rtol=1e-13)


@pytest.mark.parametrize("Tq,P,D", [(1, 0, 4), (6, 0, 4), (13, 7, 8), (4, 30, 8)])
def test_statistics_match_library_softmax(Tq, P, D):
    rng = np.random.default_rng(Tq * 10 + P)
    qb, kb = _rand_bits(rng, (3, Tq, D)), _rand_bits(rng, (3, P + Tq, D))
    A = _attention_rows(qb, kb, 0.5)                                    # [3, Tq, P+Tq]
    total = A.sum(dim=-2).numpy()
    np.testing.assert_array_equal(orc.importance_statistic(qb, kb, 0.5, orc.STAT_SUM),
                                  orc.importance_prefix(qb, kb, 0.5)[0])
    seen_by = (torch.arange(P + Tq)[None, :] <= torch.arange(Tq)[:, None] + P).sum(dim=0).numpy()
    np.testing.assert_allclose(orc.importance_statistic(qb, kb, 0.5, orc.STAT_MEAN), total / seen_by, rtol=1e-12)
    np.testing.assert_allclose(orc.importance_statistic(qb, kb, 0.5, orc.STAT_MAX), A.max(dim=-2).values.numpy(),
                               rtol=1e-12)
    beta = 0.8
    w = (1 - beta) * beta ** torch.arange(Tq - 1, -1, -1, dtype=torch.float64)   # weight of query m at the end
    want = (w[None, :, None] * A).sum(dim=-2).numpy()
    got = orc.importance_statistic(qb, kb, 0.5, orc.STAT_MOVING_AVERAGE, beta)
    np.testing.assert_allclose(got, want, rtol=1e-12)
    np.testing.assert_allclose(got.sum(-1), 1 - beta ** Tq, rtol=1e-12)          # rows of A carry unit mass
    # beta = 0 keeps only the last query's row
    np.testing.assert_allclose(orc.importance_statistic(qb, kb, 0.5, orc.STAT_MOVING_AVERAGE, 0.0),
                               A[:, -1, :].numpy(), rtol=1e-12)
    with pytest.raises(ValueError):
        orc.importance_statistic(qb, kb, 0.5, 7)


# ------------------------------------------------------------------ attention output (the forward pass of Alg. 1's input)

def test_attention_hand_example():
    rows = _rows("attention_pow2.txt")
    q = _bf16(np.array([[1.0, 0.0]] * 3).reshape(1, 3, 2))
    k = _bf16(np.array([[0.0, 5.0], [1.0, 5.0], [2.0, 5.0]]).reshape(1, 3, 2))
    v = _bf16(np.array([[1.0, 0.0], [0.0, 1.0], [4.0, -2.0]]).reshape(1, 3, 2))
    out, lse = orc.attention_prefix(q, k, v, math.log(2.0))
    want = np.array([[float(Fraction(int(a), int(b))), float(Fraction(int(c), int(d)))] for a, b, c, d, _ in rows])
    np.testing.assert_allclose(out[0], want, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(lse[0], [math.log(float(r[4])) for r in rows], atol=1e-14)


@pytest.mark.parametrize("Tq,P,D,scale", [(1, 0, 4, 1.0), (16, 0, 8, 0.5), (45, 0, 16, 0.25), (9, 13, 8, 0.4), (1, 20, 4, 1.0)])
def test_attention_matches_library_softmax(Tq, P, D, scale):
    rng = np.random.default_rng(Tq * 1000 + P * 10 + D)
    qb = _rand_bits(rng, (2, Tq, D))
    kb, vb = _rand_bits(rng, (2, P + Tq, D)), _rand_bits(rng, (2, P + Tq, D))
    out, lse = orc.attention_prefix(qb, kb, vb, scale)
    q = torch.from_numpy(orc.widen_bf16(qb))
    k = torch.from_numpy(orc.widen_bf16(kb))
    v = torch.from_numpy(orc.widen_bf16(vb))
    logits = scale * q @ k.transpose(-1, -2)
    m = torch.arange(Tq)[:, None]
    n = torch.arange(P + Tq)[None, :]
    logits = logits.masked_fill(n > m + P, float("-inf"))
    np.testing.assert_allclose(out, (torch.softmax(logits, -1) @ v).numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, -1).numpy(), rtol=1e-13, atol=1e-13)
    # the normaliser is the one the importance function reports for the same inputs
    _, lse_imp = orc.importance_prefix(qb, kb, scale)
    np.testing.assert_array_equal(lse, lse_imp)


def test_attention_zero_queries_is_running_mean_of_values():
    # uniform attention: out[m] = mean of v_0 .. v_{m+P}
    Tq, P, D = 23, 5, 8
    rng = np.random.default_rng(3)
    q = _bf16(np.zeros((1, Tq, D)))
    kb, vb = _rand_bits(rng, (1, P + Tq, D)), _rand_bits(rng, (1, P + Tq, D))
    out, lse = orc.attention_prefix(q, kb, vb, 0.9)
    v = orc.widen_bf16(vb)[0]
    want = np.cumsum(v, 0)[P:] / np.arange(P + 1, P + Tq + 1)[:, None]
    np.testing.assert_allclose(out[0], want, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(lse[0], np.log(np.arange(P + 1, P + Tq + 1)), atol=1e-13)


def test_attention_invariants():
    Tq, P, D = 31, 7, 8
    rng = np.random.default_rng(11)
    qb = _rand_bits(rng, (1, Tq, D), 2.0)
    kb, vb = _rand_bits(rng, (1, P + Tq, D)), _rand_bits(rng, (1, P + Tq, D))
    out, _ = orc.attention_prefix(qb, kb, vb, 0.5)
    v = orc.widen_bf16(vb)[0]
    # a convex combination of the visible value rows, coordinate by coordinate
    for m in range(Tq):
        vis = v[: m + P + 1]
        assert np.all(out[0, m] <= vis.max(0) + 1e-12) and np.all(out[0, m] >= vis.min(0) - 1e-12)
    # constant values come out unchanged whatever the attention is
    const = _bf16(np.tile(np.array([1.5, -2.0, 0.25, 3.0, 0.0, 1.0, -1.0, 8.0], np.float32), (1, P + Tq, 1)))
    out_c, _ = orc.attention_prefix(qb, kb, const, 0.5)
    np.testing.assert_allclose(out_c[0], np.tile(orc.widen_bf16(const)[0, :1], (Tq, 1)), rtol=1e-13)
    # summing the output rows weights every value row by the importance it received (Eq. 1's column sums)
    scores, _ = orc.importance_prefix(qb, kb, 0.5)
    np.testing.assert_allclose(out[0].sum(0), scores[0] @ v, rtol=1e-12, atol=1e-12)
    # a change to a key or value the query cannot see changes nothing for that query
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[0, P + 10:] = _rand_bits(rng, (Tq - 10, D))
    vb2[0, P + 10:] = _rand_bits(rng, (Tq - 10, D))
    out2, _ = orc.attention_prefix(qb, kb2, vb2, 0.5)
    np.testing.assert_array_equal(out2[0, :10], out[0, :10])
