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


def run_timed_configuration(w, sample_units):
    """Every problem of a configuration, with its full decode length, through the same calls and launch
    shapes the benchmark times (one CTA per unit in the decode loop, many waves, overlapped steps; the
    selection and merge grids over every unit). Properties that hold for any input are checked on all
    units on the device; the sampled (n, h) units are recomputed by the oracle one by one."""
    import os
    threads = min(16, os.cpu_count() or 8)
    Qb, Kb, Vb = wl.prompt(w, threads=threads)
    N, H, T, D = Qb.shape
    steps = w.decode_steps
    sess = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    C = sess.n_keep
    Q, K, V = dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)
    sess.compress(Q, K, V)
    assert ec.ec_device_status(sess.ws_imp) == ec.EC_OK
    assert ec.ec_decode_splits(sess.cache) == 1                 # the unsplit path, as timed
    del Q
    sc, an = sess.scores, sess.anchor_pos.long()

    # properties of every unit, evaluated on the device
    assert torch.allclose(sc.double().sum(-1), torch.full((N, H), float(T), dtype=torch.float64, device="cuda"), rtol=1e-3)
    assert bool((sc > 0).all()) and bool((sc[..., 0] >= 1.0 - 1e-3).all())
    assert bool((an[..., 1:] > an[..., :-1]).all()) and bool((an[..., 0] == 0).all()) and bool((an[..., -1] == T - 1).all())
    kth = torch.sort(sc, dim=-1, descending=True).values[..., C - 1]
    picked = torch.gather(sc, -1, an)[..., 1:-1]
    assert bool((picked >= kth[..., None] * (1 - 1e-6)).all())   # nothing below the threshold is kept
    # Eq. 3 conserves mass: sum_k |B_k| * mean_k = sum_t row_t, for K and V (bf16 rounding of the means
    # bounds the difference by T * 2^-9 * max|row|)
    mid = (an[..., :-1] + an[..., 1:]) // 2
    hi = torch.cat([mid, torch.full_like(an[..., :1], T - 1)], -1)
    lo = torch.cat([torch.zeros_like(an[..., :1]), mid + 1], -1)
    size = (hi - lo + 1).float()
    assert bool((size >= 1).all()) and bool((size.sum(-1) == T).all())
    for X, Xc in ((K, sess.Kc), (V, sess.Vc)):
        for n0 in range(0, N, 32):                               # chunks keep the fp32 temporaries small
            sl = slice(n0, min(n0 + 32, N))
            total = X[sl].float().sum(2)
            back = (Xc[sl, :, :C].float() * size[sl, ..., None]).sum(2)
            bound = T * 2.0 ** -8 * X[sl].float().abs().amax(2) + 1e-3
            assert bool(((total - back).abs() <= bound).all())
    Kc0 = {u: host_f64(sess.Kc[u[0], u[1]]) for u in sample_units}
    Vc0 = {u: host_f64(sess.Vc[u[0], u[1]]) for u in sample_units}
    scores = {u: sc[u[0], u[1]].cpu().double().numpy() for u in sample_units}
    anchors = {u: sess.anchor_pos[u[0], u[1]].cpu().numpy() for u in sample_units}
    del K, V

    qb, kb, vb = wl.decode_inputs(w, steps, threads=threads)
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    out = torch.empty_like(q)
    slots = sess.decode(q, k, v, out, want_slots=True)
    torch.cuda.synchronize()
    assert slots == [(C - w.offset) + (s % w.offset) for s in range(steps)]
    assert sess.cache.len == C and sess.cache.step == steps and ec.ec_decode_splits(sess.cache) == 1
    assert bool(torch.isfinite(out.float()).all())
    # the output of a step is a convex combination of the value rows it attended to
    vmax = torch.maximum(sess.Vc.float().amax(2), v.float().amax(0))
    vmin = torch.minimum(sess.Vc.float().amin(2), v.float().amin(0))
    tail = out[-1].float()
    assert bool((tail <= vmax + 2e-2 + 2.0 ** -8 * vmax.abs()).all()) and bool((tail >= vmin - 2e-2 - 2.0 ** -8 * vmin.abs()).all())

    # sampled units against the oracle, importance of all of them in one (threaded) oracle call
    o_scores_all, _ = orc.importance(np.stack([Qb[n, h] for n, h in sample_units]),
                                     np.stack([Kb[n, h] for n, h in sample_units]), w.scale)
    for i, (n, h) in enumerate(sample_units):
        o_scores = o_scores_all[i][None]
        assert (np.abs(scores[(n, h)] - o_scores[0]) <= SCORE_RTOL * np.abs(o_scores[0])).all(), (n, h)
        o_anch = orc.select(o_scores, C, True)
        if not (o_anch[0] == anchors[(n, h)]).all():
            s = o_scores[0].copy()
            s[0] = s[-1] = np.inf
            kth_o = np.sort(s)[::-1][C - 1]
            diff = np.setxor1d(o_anch[0], anchors[(n, h)])
            assert (np.abs(s[diff] - kth_o) <= 1e-4 * kth_o).all(), (n, h, diff)
            o_anch = anchors[(n, h)][None]          # both selections are valid: follow the GPU's
        lo_o, hi_o = orc.buckets(o_anch, T)
        o_K, o_V = orc.merge(Kb[n, h][None], lo_o, hi_o), orc.merge(Vb[n, h][None], lo_o, hi_o)
        assert close_bf16(Kc0[(n, h)][:C], o_K[0]).all() and close_bf16(Vc0[(n, h)][:C], o_V[0]).all(), (n, h)
        queue = orc.DecodeQueue(orc.widen_bf16(orc.round_bf16(o_K)), orc.widen_bf16(orc.round_bf16(o_V)), cap=C + 1)
        out_u = host_f64(out[:, n, h])
        for s_ in range(steps):
            want, pos, _ = queue.step(qb[s_, n, h][None], kb[s_, n, h][None], vb[s_, n, h][None], w.scale,
                                      policy=orc.POLICY_FIXED, budget=C, offset=w.offset)
            assert pos == C - w.offset
            assert close_bf16(out_u[s_], want[0]).all(), (n, h, s_)
        # the cache after the last step holds the oracle's queue: the merged prompt rows that never
        # moved, and, bit for bit, the `offset` newest generated rows in the ring (rotated)
        Kend, Vend = host_f64(sess.Kc[n, h]), host_f64(sess.Vc[n, h])
        base = C - w.offset
        assert close_bf16(Kend[:base], queue.K[0, :base]).all() and close_bf16(Vend[:base], queue.V[0, :base]).all()
        assert sorted(Kend[base:C].tolist()) == sorted(queue.K[0, base:C].tolist()), (n, h)
        assert sorted(Vend[base:C].tolist()) == sorted(queue.V[0, base:C].tolist()), (n, h)


def test_7b_batch8_every_problem_as_timed():
    w = wl.WORKLOADS["llava7b_b8"]           # 8192 units x 256 kept rows, 512 steps: many waves of one-CTA units
    run_timed_configuration(w, [(0, 0), (100, 16), (255, 31), (131, 7)])


def test_long_context_every_problem_as_timed():
    w = wl.WORKLOADS["long8k"]               # 2048 units x 820 kept rows, 2048 steps
    run_timed_configuration(w, [(0, 3), (37, 30), (63, 31)])


def test_13b_every_problem_as_timed():
    import dataclasses
    w = dataclasses.replace(wl.WORKLOADS["llava13b_b4"], keep_ratios=(0.25,))   # 6400 units x 512 kept rows, 1024 steps
    run_timed_configuration(w, [(3, 0), (150, 39), (80, 20)])


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
