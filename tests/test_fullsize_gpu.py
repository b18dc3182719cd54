"""Parity at the sizes and in the launch configuration the benchmark times: the whole
llava7b_b1 workload (32 layers x 32 heads, 640-token prompt, 512 decode steps through the
native step loop), checked on sampled units the oracle computes one by one and on properties
that hold for every unit; plus full-length (8192-token) units of the long-context workload."""
import numpy as np
import pytest
import torch

from oracle import ec_oracle as orc
from paper_2407_18121_b200 import binding as ec
from paper_2407_18121_b200 import workloads as wl
from paper_2407_18121_b200.session import ElasticCacheSession
from helpers import BF16_ATOL, BF16_RTOL, SCORE_RTOL, dev_bf16, host_f64

pytestmark = pytest.mark.gpu


def close_bf16(got, want):
    return np.abs(got - want) <= BF16_ATOL + BF16_RTOL * np.abs(want)


def run_workload(w, problems, sample_units, steps):
    """GPU: all listed problems at once, exactly as bench.py drives it. Oracle: sampled (n, h) units."""
    Qb, Kb, Vb = wl.prompt(w, problems)
    N, H, T, D = Qb.shape
    sess = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    C = sess.n_keep
    Q, K, V = dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)
    sess.compress(Q, K, V)
    assert ec.ec_device_status(sess.ws_imp) == ec.EC_OK
    scores = sess.scores.cpu().double().numpy()
    anchors = sess.anchor_pos.cpu().numpy()
    Kc0, Vc0 = host_f64(sess.Kc), host_f64(sess.Vc)

    # properties of every unit
    np.testing.assert_allclose(scores.sum(-1), T, rtol=1e-3)            # rows of A sum to one
    assert (scores > 0).all() and (scores[..., 0] >= 1.0 - 1e-3).all()
    assert (np.diff(anchors, axis=-1) > 0).all() and anchors.min() == 0 and anchors.max() == T - 1
    assert (anchors[..., 0] == 0).all() and (anchors[..., -1] == T - 1).all()   # protected ends
    kth = np.sort(scores, axis=-1)[..., ::-1][..., C - 1]
    picked = np.take_along_axis(scores, anchors.astype(np.int64), -1)[..., 1:-1]
    assert (picked >= kth[..., None] * (1 - 1e-6)).all()                 # nothing below the threshold is kept

    qb, kb, vb = wl.decode_inputs(w, steps, problems)
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    out = torch.empty_like(q)
    slots = sess.decode(q, k, v, out, want_slots=True)
    torch.cuda.synchronize()
    assert slots == [(C - w.offset) + (s % w.offset) for s in range(steps)]
    assert sess.cache.len == C and sess.cache.step == steps
    out_h = host_f64(out)
    assert np.isfinite(out_h).all()

    # sampled units against the oracle
    for (n, h) in sample_units:
        o_scores, _ = orc.importance(Qb[n, h][None], Kb[n, h][None], w.scale)
        assert (np.abs(scores[n, h] - o_scores[0]) <= SCORE_RTOL * np.abs(o_scores[0])).all(), (n, h)
        o_anch = orc.select(o_scores, C, True)
        if not (o_anch[0] == anchors[n, h]).all():
            s = o_scores[0].copy()
            s[0] = s[-1] = np.inf
            kth_o = np.sort(s)[::-1][C - 1]
            diff = np.setxor1d(o_anch[0], anchors[n, h])
            assert (np.abs(s[diff] - kth_o) <= 1e-4 * kth_o).all(), (n, h, diff)
            o_anch = anchors[n, h][None]          # both selections are valid: follow the GPU's
        lo, hi = orc.buckets(o_anch, T)
        o_K, o_V = orc.merge(Kb[n, h][None], lo, hi), orc.merge(Vb[n, h][None], lo, hi)
        assert close_bf16(Kc0[n, h, :C], o_K[0]).all() and close_bf16(Vc0[n, h, :C], o_V[0]).all(), (n, h)
        queue = orc.DecodeQueue(orc.widen_bf16(orc.round_bf16(o_K)), orc.widen_bf16(orc.round_bf16(o_V)), cap=C + 1)
        for s_ in range(steps):
            want, pos, _ = queue.step(qb[s_, n, h][None], kb[s_, n, h][None], vb[s_, n, h][None], w.scale,
                                      policy=orc.POLICY_FIXED, budget=C, offset=w.offset)
            assert pos == C - w.offset
            assert close_bf16(out_h[s_, n, h], want[0]).all(), (n, h, s_)
    return sess


def test_benchmark_workload_full_size():
    w = wl.WORKLOADS["llava7b_b1"]
    sample = [(0, 0), (0, 31), (13, 17), (31, 0), (31, 31), (20, 5)]
    run_workload(w, list(range(w.N)), sample, w.decode_steps)


def test_long_context_units_full_length():
    w = wl.WORKLOADS["long8k"]
    run_workload(w, [0, 37], [(0, 3), (1, 30)], 40)


@pytest.mark.parametrize("ratio", [0.1, 0.25, 0.5, 0.75])
def test_13b_shapes_full_length_ratio_sweep(ratio):
    import dataclasses
    w = dataclasses.replace(wl.WORKLOADS["llava13b_b4"], keep_ratios=(ratio,))   # 40 heads, T = 2048
    run_workload(w, [3, 150], [(0, 0), (1, 39)], 20)


def test_7b_batch8_shapes_full_length():
    w = wl.WORKLOADS["llava7b_b8"]           # T = 1024, ratio 0.25 -> 256 kept rows
    run_workload(w, [0, 100, 255], [(0, 0), (1, 16), (2, 31)], 40)


def test_qwenvl_shapes_full_size():
    w = wl.WORKLOADS["qwenvl7b_b1"]          # T = 320 (2.5 tiles), 160 kept rows, recent distance 25
    run_workload(w, list(range(w.N)), [(0, 0), (7, 19), (31, 31)], 60)


def test_longest_supported_prompt():
    """T = 16384 (the documented maximum), one unit: 128 tiles per pass in the importance kernels,
    64 KB of keys in the selection kernel's shared memory, 64 slices in the merge kernel."""
    rng = np.random.default_rng(16384)
    N, H, T, D, ratio = 1, 1, 16384, 64, 0.1
    Qb = wl.to_bf16_bits(rng.standard_normal((N, H, T, D)).astype(np.float32))
    Kb = wl.to_bf16_bits(rng.standard_normal((N, H, T, D)).astype(np.float32))
    Vb = wl.to_bf16_bits(rng.standard_normal((N, H, T, D)).astype(np.float32))
    sess = ElasticCacheSession(N, H, T, D, ratio, 16, 0.125)
    sess.compress(dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb))
    assert ec.ec_device_status(sess.ws_imp) == ec.EC_OK
    C = sess.n_keep
    assert C == orc.keep_count(T, ratio) == 1639
    o_scores, _ = orc.importance(Qb, Kb, 0.125)
    scores = sess.scores.cpu().double().numpy()
    assert (np.abs(scores - o_scores) <= SCORE_RTOL * np.abs(o_scores)).all()
    o_anch = orc.select(o_scores, C, True)
    anchors = sess.anchor_pos.cpu().numpy()
    if not (anchors == o_anch).all():
        s = o_scores[0, 0].copy()
        s[0] = s[-1] = np.inf
        kth = np.sort(s)[::-1][C - 1]
        diff = np.setxor1d(anchors[0, 0], o_anch[0, 0])
        assert (np.abs(s[diff] - kth) <= 1e-4 * kth).all()
        o_anch = anchors
    lo, hi = orc.buckets(o_anch, T)
    assert close_bf16(host_f64(sess.Kc), orc.merge(Kb, lo, hi)).all()
    assert close_bf16(host_f64(sess.Vc), orc.merge(Vb, lo, hi)).all()


def test_reruns_are_bit_identical():
    """No kernel uses floating-point atomics or a schedule-dependent reduction order."""
    w = wl.WORKLOADS["llava7b_b1"]
    Qb, Kb, Vb = wl.prompt(w, [4, 9])
    qb, kb, vb = wl.decode_inputs(w, 20, [4, 9])
    N, H, T, D = Qb.shape
    Q, K, V, q, k, v = (dev_bf16(x) for x in (Qb, Kb, Vb, qb, kb, vb))
    results = []
    for _ in range(2):
        sess = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
        sess.compress(Q, K, V)
        out = torch.empty_like(q)
        sess.decode(q, k, v, out)
        torch.cuda.synchronize()
        results.append((sess.scores.clone(), sess.anchor_pos.clone(), sess.Kc.clone(), sess.Vc.clone(), out))
    for a, b in zip(*results):
        assert torch.equal(a, b)
