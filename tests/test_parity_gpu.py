"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded bf16 inputs. Oracle inputs never come from the GPU: stage tests feed the
GPU with the oracle's own intermediate results."""
import math

import numpy as np
import pytest
import torch

from oracle import ec_oracle as orc
from paper_2407_18121_b200 import binding as ec
from paper_2407_18121_b200 import workloads as wl
from helpers import (SCORE_RTOL, Guarded, assert_bf16_close, assert_rel_close, dev_bf16, host_bits, host_f64,
                     scratch)

pytestmark = pytest.mark.gpu


def rand_bits(rng, shape, sigma=1.0):
    return wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.float32(sigma))


# ---------------------------------------------------------------- stage runners

def gpu_importance(Qb, Kb, scale, want_lse=True):
    N, H, T, D = Qb.shape
    Q, K = dev_bf16(Qb), dev_bf16(Kb)
    scores = Guarded((N, H, T), torch.float32, fill=float("nan"))
    lse = Guarded((N, H, T), torch.float32, fill=float("nan")) if want_lse else None
    ws = scratch(ec.ec_importance_workspace(N, H, T, D))
    ec.ec_importance(Q, K, scores.t, lse.t if lse else None, scale, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    scores.check("scores")
    if lse:
        lse.check("lse")
    return scores.t, (lse.t if lse else None)


def gpu_select_merge(Kb, Vb, scores_f32, n_keep, population, protect, cap=None):
    N, H, T, D = Kb.shape
    cap = n_keep if cap is None else cap
    K, V = dev_bf16(Kb), dev_bf16(Vb)
    s = torch.from_numpy(np.ascontiguousarray(scores_f32, np.float32)).cuda()
    Kc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    Vc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    anchors = Guarded((N, H, n_keep), torch.int32, fill=-7)
    blen = Guarded((N, H, n_keep), torch.int32, fill=-7)
    ws = scratch(ec.ec_select_merge_workspace(N, H, T, D, n_keep, population))
    ec.ec_select_merge(K, V, s, n_keep, population, protect, Kc.t, Vc.t, anchors.t, blen.t, ws)
    for g, name in ((Kc, "Kc"), (Vc, "Vc"), (anchors, "anchor_pos"), (blen, "bucket_len")):
        g.check(name)
    return Kc.t, Vc.t, anchors.t, blen.t


def check_anchor_sets(gpu_anchors, oracle_anchors, scores64, n_keep, protect, band=1e-4):
    """Index sets must be equal, except for positions whose score lies within `band` (relative)
    of the n_keep-th largest score: there either choice is a correct answer."""
    ga = gpu_anchors.cpu().numpy()
    T = scores64.shape[-1]
    ga2 = ga.reshape(-1, n_keep)
    oa2 = oracle_anchors.reshape(-1, n_keep)
    sc2 = scores64.reshape(-1, T)
    exact = 0
    for u in range(ga2.shape[0]):
        assert (np.diff(ga2[u]) > 0).all(), "anchors must be strictly ascending"
        assert ga2[u].min() >= 0 and ga2[u].max() < T
        if (ga2[u] == oa2[u]).all():
            exact += 1
            continue
        s = sc2[u].copy()
        if protect:
            s[0] = np.inf
            if n_keep >= 2:
                s[-1] = np.inf
        kth = np.sort(s)[::-1][n_keep - 1]
        diff = np.setxor1d(ga2[u], oa2[u])
        assert (np.abs(s[diff] - kth) <= band * abs(kth)).all(), \
            f"unit {u}: anchor sets differ outside the tie band at positions {diff}"
    return exact, ga2.shape[0]


def anchors_to_merge_on(gpu_anchors, oracle_anchors):
    """Anchor sets the oracle's merge is run on: the oracle's own, except for units where the two
    sides differ inside the tie band (already verified by check_anchor_sets): there both selections
    are valid answers and the GPU's merge can only be checked on the set it chose."""
    ga = gpu_anchors.cpu().numpy()
    same = (ga == oracle_anchors).all(axis=-1, keepdims=True)
    return np.where(same, oracle_anchors, ga)


# ---------------------------------------------------------------- importance

@pytest.mark.parametrize("N,H,T,D", [(1, 1, 1, 64), (1, 2, 2, 128), (2, 2, 127, 64), (1, 3, 129, 128),
                                     (1, 2, 255, 128), (2, 1, 256, 64), (1, 2, 640, 128), (1, 1, 300, 64)])
def test_importance_random(N, H, T, D):
    rng = np.random.default_rng(T * 7 + D)
    Qb, Kb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    scale = 1.0 / math.sqrt(D)
    want, want_lse = orc.importance(Qb, Kb, scale)
    got, got_lse = gpu_importance(Qb, Kb, scale)
    assert_rel_close(got, want, SCORE_RTOL, what="scores")
    assert_rel_close(got_lse, want_lse, 1e-3, atol=1e-3, what="lse")
    np.testing.assert_allclose(host_f64(got).sum(-1), T, rtol=1e-3)      # rows of A sum to one


def test_importance_peaked_logits_and_no_lse_output():
    # large logits: the row maximum must be subtracted or exp overflows
    rng = np.random.default_rng(3)
    Qb, Kb = rand_bits(rng, (1, 2, 200, 128), 3.0), rand_bits(rng, (1, 2, 200, 128), 3.0)
    want, _ = orc.importance(Qb, Kb, 1.0)
    got, none = gpu_importance(Qb, Kb, 1.0, want_lse=False)
    assert none is None
    assert_rel_close(got, want, SCORE_RTOL, atol=1e-30, what="scores (peaked)")


@pytest.mark.parametrize("name", ["tiny", "llava7b_b1", "long8k"])
def test_importance_on_workload_recipes(name):
    w = wl.WORKLOADS[name]
    if name == "llava7b_b1":
        Qb, Kb, _ = wl.prompt(w, [0, 31])
        Qb, Kb = Qb[:, :4], Kb[:, :4]
    elif name == "long8k":
        Qb, Kb, _ = wl.prompt(w, [5])
        Qb, Kb = Qb[:, :2, :1536], Kb[:, :2, :1536]      # several tiles of the recipe, oracle-sized
    else:
        Qb, Kb, _ = wl.prompt(w)
    Qb, Kb = np.ascontiguousarray(Qb), np.ascontiguousarray(Kb)
    want, want_lse = orc.importance(Qb, Kb, w.scale)
    got, got_lse = gpu_importance(Qb, Kb, w.scale)
    assert_rel_close(got, want, SCORE_RTOL, what=f"scores[{name}]")
    assert_rel_close(got_lse, want_lse, 1e-3, atol=1e-3, what=f"lse[{name}]")


def test_importance_is_deterministic():
    rng = np.random.default_rng(8)
    Qb, Kb = rand_bits(rng, (2, 3, 333, 128)), rand_bits(rng, (2, 3, 333, 128))
    a, _ = gpu_importance(Qb, Kb, 0.1)
    b, _ = gpu_importance(Qb, Kb, 0.1)
    assert torch.equal(a, b)


# ---------------------------------------------------------------- selection + merge

@pytest.mark.parametrize("population", [ec.EC_PER_HEAD, ec.EC_LAYER_SHARED])
@pytest.mark.parametrize("protect", [False, True])
@pytest.mark.parametrize("N,H,T,D,n_keep", [(1, 1, 1, 64, 1), (1, 2, 2, 64, 1), (2, 3, 130, 128, 65),
                                            (1, 4, 257, 64, 26), (2, 2, 640, 128, 320), (1, 2, 1000, 128, 1),
                                            (1, 2, 300, 128, 299), (1, 1, 2048, 128, 205)])
def test_select_merge_from_oracle_scores(N, H, T, D, n_keep, population, protect):
    rng = np.random.default_rng(T + n_keep)
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    # heavy-tailed positive scores, as column sums of attention are; fp32-exact so both sides rank
    # the very same numbers
    s32 = (rng.random((N, H, T)) ** 4 * 5 + 1e-3).astype(np.float32)
    s64 = s32.astype(np.float64)
    if population == ec.EC_LAYER_SHARED:
        rank64 = np.repeat(orc.layer_mean(s64)[:, None, :], H, axis=1)
    else:
        rank64 = s64
    want_anchors = orc.select(rank64, n_keep, protect)
    Kc, Vc, anchors, blen = gpu_select_merge(Kb, Vb, s32, n_keep, population, protect)
    exact, total = check_anchor_sets(anchors, want_anchors, rank64, n_keep, protect)
    if population == ec.EC_PER_HEAD:
        assert exact == total                       # same fp32 numbers on both sides: bit-exact sets
    ga = anchors.cpu().numpy()
    if population == ec.EC_LAYER_SHARED:
        assert (ga == ga[:, :1]).all()              # every head of a problem shares the anchors
    lo, hi = orc.buckets(anchors_to_merge_on(anchors, want_anchors), T)
    np.testing.assert_array_equal(blen.cpu().numpy(), hi - lo + 1)
    assert_bf16_close(Kc, orc.merge(Kb, lo, hi), "merged K")
    assert_bf16_close(Vc, orc.merge(Vb, lo, hi), "merged V")


def test_keep_everything_is_the_identity():
    rng = np.random.default_rng(21)
    N, H, T, D = 2, 3, 193, 128
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    s32 = rng.random((N, H, T)).astype(np.float32)
    Kc, Vc, anchors, blen = gpu_select_merge(Kb, Vb, s32, T, ec.EC_PER_HEAD, True)
    np.testing.assert_array_equal(host_bits(Kc), Kb)          # bit-identical cache
    np.testing.assert_array_equal(host_bits(Vc), Vb)
    assert (anchors.cpu().numpy() == np.arange(T)).all() and (blen.cpu().numpy() == 1).all()


def test_exact_ties_go_to_the_lower_position():
    N, H, T, D = 1, 2, 96, 64
    rng = np.random.default_rng(5)
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    s32 = rng.integers(1, 4, size=(N, H, T)).astype(np.float32)       # only three distinct values
    for n_keep in (1, 10, 48, 95):
        want = orc.select(s32.astype(np.float64), n_keep, False)
        _, _, anchors, _ = gpu_select_merge(Kb, Vb, s32, n_keep, ec.EC_PER_HEAD, False)
        np.testing.assert_array_equal(anchors.cpu().numpy(), want)


def test_cap_larger_than_keep_leaves_tail_rows_untouched():
    rng = np.random.default_rng(6)
    N, H, T, D, n_keep, cap = 1, 2, 100, 128, 30, 47
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    s32 = rng.random((N, H, T)).astype(np.float32)
    Kc, Vc, anchors, _ = gpu_select_merge(Kb, Vb, s32, n_keep, ec.EC_PER_HEAD, False, cap=cap)
    assert torch.isnan(Kc[:, :, n_keep:].float()).all() and torch.isnan(Vc[:, :, n_keep:].float()).all()
    want_anchors = orc.select(s32.astype(np.float64), n_keep, False)
    np.testing.assert_array_equal(anchors.cpu().numpy(), want_anchors)
    lo, hi = orc.buckets(want_anchors, T)
    assert_bf16_close(Kc[:, :, :n_keep].contiguous(), orc.merge(Kb, lo, hi), "merged K")


# ---------------------------------------------------------------- decode + fixed-point eviction

def run_decode_case(N, H, D, C, cap, len0, offset, steps, scale, seed, sigma_k=1.0):
    """Cache contents come from the oracle side (random bf16 rows); both sides run `steps` steps."""
    rng = np.random.default_rng(seed)
    K0b, V0b = rand_bits(rng, (N, H, len0, D), sigma_k), rand_bits(rng, (N, H, len0, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=max(C, len0) + 1)
    Kc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    Vc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    Kc.t[:, :, :len0] = dev_bf16(K0b)
    Vc.t[:, :, :len0] = dev_bf16(V0b)
    cache = ec.ec_cache_init(Kc.t, Vc.t, len0, C, offset)
    ws = scratch(ec.ec_decode_workspace(cache))
    slot_ids = list(range(len0)) + [-1] * (cap - len0)        # identity held by each physical slot
    evictions = 0
    for s in range(steps):
        qb, kb, vb = rand_bits(rng, (N, H, D)), rand_bits(rng, (N, H, D), sigma_k), rand_bits(rng, (N, H, D))
        len_before = cache.len
        want, pos, ident = queue.step(qb, kb, vb, scale, policy=orc.POLICY_FIXED, budget=C, offset=offset)
        out = Guarded((N, H, D), torch.bfloat16, fill=float("nan"))
        ev, slot = ec.ec_decode_step(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, scale, out.t, ws)
        out.check("out")
        assert_bf16_close(out.t, want, f"decode out, step {s}")
        if len_before < C:
            assert ev == -1 and pos == -1 and slot == len_before
        else:
            assert pos == C - offset                                 # the fixed truncation location
            assert ev == slot == (C - offset) + (evictions % offset)  # ring of `offset` slots
            assert slot_ids[ev] == ident                              # the same row leaves on both sides
            evictions += 1
        slot_ids[slot] = queue.next_id - 1
        assert cache.len == queue.len and cache.step == s + 1
        assert sorted(slot_ids[:cache.len]) == sorted(queue.identities().tolist())
    Kc.check("Kc")
    Vc.check("Vc")
    # the device cache holds exactly the oracle queue's rows (as a set; order is physical)
    Kdev = host_f64(Kc.t[:, :, :cache.len])
    ids = queue.identities().tolist()
    for j, ident in enumerate(ids):
        phys = slot_ids.index(ident)
        np.testing.assert_array_equal(Kdev[:, :, phys], queue.K[:, j].reshape(N, H, D))
    return cache


@pytest.mark.parametrize("N,H,D,C,offset,steps", [
    (1, 8, 64, 128, 16, 40),        # few units, short cache: one CTA per unit
    (1, 8, 64, 600, 16, 12),        # few units, longer cache: the rows of a unit are split over three CTAs
    (1, 2, 128, 70, 25, 60),        # the paper's recent distance of 25
    (20, 32, 128, 96, 16, 20),      # many units: one CTA per unit
    (3, 5, 64, 33, 1, 5),           # offset 1: only the newest row is protected
    (2, 2, 128, 9, 8, 20),          # offset = budget - 1: only the first row is protected
])
def test_decode_at_budget(N, H, D, C, offset, steps):
    run_decode_case(N, H, D, C, C, C, offset, steps, 1.0 / math.sqrt(D), seed=C + offset)


def test_decode_below_budget_grows_then_evicts():
    cache = run_decode_case(2, 4, 128, 40, 48, 30, 6, 25, 0.1, seed=77)
    assert cache.len == 40


def test_decode_from_empty_cache():
    # len 0: the first step attends to the new row only, so out == v_new exactly
    N, H, D = 1, 3, 64
    rng = np.random.default_rng(1)
    Kc = torch.zeros((N, H, 8, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    cache = ec.ec_cache_init(Kc, Vc, 0, 4, 2)
    ws = scratch(ec.ec_decode_workspace(cache))
    qb, kb, vb = rand_bits(rng, (N, H, D)), rand_bits(rng, (N, H, D)), rand_bits(rng, (N, H, D))
    out = torch.empty((N, H, D), dtype=torch.bfloat16, device="cuda")
    ev, slot = ec.ec_decode_step(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, 1.0, out, ws)
    assert (ev, slot, cache.len) == (-1, 0, 1)
    np.testing.assert_array_equal(host_bits(out), vb)
    np.testing.assert_array_equal(host_bits(Kc[:, :, 0]), kb)


def test_decode_peaked_logits():
    run_decode_case(1, 4, 128, 64, 64, 64, 16, 6, 1.0, seed=9, sigma_k=3.0)


def test_decode_steps_native_loop_matches_single_steps():
    rng = np.random.default_rng(4)
    N, H, D, C, d, S = 2, 3, 128, 50, 16, 37
    K0, V0 = dev_bf16(rand_bits(rng, (N, H, C, D))), dev_bf16(rand_bits(rng, (N, H, C, D)))
    q, k, v = (dev_bf16(rand_bits(rng, (S, N, H, D))) for _ in range(3))
    Ka, Va, Kb_, Vb_ = K0.clone(), V0.clone(), K0.clone(), V0.clone()
    ca, cb = ec.ec_cache_init(Ka, Va, C, C, d), ec.ec_cache_init(Kb_, Vb_, C, C, d)
    ws = scratch(ec.ec_decode_workspace(ca))
    out_a = torch.empty((S, N, H, D), dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty_like(out_a)
    slots_a = [ec.ec_decode_step(q[s], k[s], v[s], ca, 0.2, out_a[s], ws)[0] for s in range(S)]
    slots_b = ec.ec_decode_steps(q, k, v, cb, 0.2, out_b, ws, want_slots=True)
    assert slots_a == slots_b == [(C - d) + (s % d) for s in range(S)]
    assert torch.equal(out_a, out_b) and torch.equal(Ka, Kb_) and torch.equal(Va, Vb_)
    assert (cb.len, cb.ring_head, cb.step) == (C, S % d, S)


@pytest.mark.parametrize("N,H,D,C,len0,offset,steps", [
    (1, 8, 128, 600, 200, 16, 420),     # grows from one CTA per unit to three, then evicts at the budget
    (1, 3, 64, 700, 700, 25, 30),       # three CTAs per unit from the first step on
    (4, 32, 128, 512, 512, 16, 24),     # 128 units: three CTAs each, consecutive steps overlap
])
def test_split_units_with_a_dirty_workspace(N, H, D, C, len0, offset, steps):
    """Few units: a unit's rows are shared by several CTAs and the last one to arrive merges their
    partial results. The workspace starts full of ones (arrival counters included), is reused by
    single-step calls and by the native loop, and the outputs must match the oracle throughout."""
    rng = np.random.default_rng(len0 + steps)
    scale = 1.0 / math.sqrt(D)
    K0b, V0b = rand_bits(rng, (N, H, len0, D)), rand_bits(rng, (N, H, len0, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=C + 1)
    Kc = torch.zeros((N, H, C, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    Kc[:, :, :len0], Vc[:, :, :len0] = dev_bf16(K0b), dev_bf16(V0b)
    cache = ec.ec_cache_init(Kc, Vc, len0, C, offset)
    ws = torch.full((ec.ec_decode_workspace(cache),), 0xFF, dtype=torch.uint8, device="cuda")
    qb, kb, vb = (rand_bits(rng, (steps, N, H, D)) for _ in range(3))
    want = np.stack([queue.step(qb[s], kb[s], vb[s], scale, policy=orc.POLICY_FIXED, budget=C, offset=offset)[0]
                     for s in range(steps)])
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    out = torch.empty((steps, N, H, D), dtype=torch.bfloat16, device="cuda")
    single = steps // 3                                       # first third: one call per step
    for s in range(single):
        ec.ec_decode_step(q[s], k[s], v[s], cache, scale, out[s], ws)
    ws.fill_(0xFF)                                            # dirty again before the native loop
    ec.ec_decode_steps(q[single:], k[single:], v[single:], cache, scale, out[single:], ws)
    assert cache.len == queue.len and cache.step == steps
    for s in range(steps):
        assert_bf16_close(out[s], want[s], f"split decode, step {s}")


# ---------------------------------------------------------------- the whole path

@pytest.mark.parametrize("name,population", [("tiny", ec.EC_PER_HEAD), ("tiny", ec.EC_LAYER_SHARED),
                                             ("llava7b_b1", ec.EC_PER_HEAD)])
def test_whole_path_on_workload(name, population):
    """importance -> select/merge -> decode loop entirely on the GPU, against the oracle chain."""
    w = wl.WORKLOADS[name]
    if name == "llava7b_b1":
        problems, heads, steps = [7], 3, 24
    else:
        problems, heads, steps = [0], w.heads, w.decode_steps
    Qb, Kb, Vb = (np.ascontiguousarray(x[:, :heads]) for x in wl.prompt(w, problems))
    N, H, T, D = Qb.shape
    C = ec.ec_keep_count(T, w.keep_ratio)
    assert C == orc.keep_count(T, w.keep_ratio)

    o_scores, _ = orc.importance(Qb, Kb, w.scale)
    rank = o_scores if population == ec.EC_PER_HEAD else np.repeat(orc.layer_mean(o_scores)[:, None], H, 1)
    o_anchors = orc.select(rank, C, True)

    Q, K, V = dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)
    scores = torch.empty((N, H, T), dtype=torch.float32, device="cuda")
    ws_i = scratch(ec.ec_importance_workspace(N, H, T, D))
    ec.ec_importance(Q, K, scores, None, w.scale, ws_i)
    Kc = torch.empty((N, H, C, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.empty_like(Kc)
    anchors = torch.empty((N, H, C), dtype=torch.int32, device="cuda")
    ws_m = scratch(ec.ec_select_merge_workspace(N, H, T, D, C, population))
    ec.ec_select_merge(K, V, scores, C, population, True, Kc, Vc, anchors, None, ws_m)
    assert_rel_close(scores, o_scores, SCORE_RTOL, what="scores")
    check_anchor_sets(anchors, o_anchors, rank, C, True)
    if name == "tiny" and population == ec.EC_PER_HEAD:
        # a boosted key draws attention from every later query, so those that are not close to
        # the end of the prompt (where few queries remain to look at them) must all be anchors
        knorm = np.linalg.norm(wl.bf16_bits_to_f64(Kb), axis=-1)
        for h in range(H):
            heavy = np.argsort(knorm[0, h])[-4:]
            heavy = heavy[heavy < (3 * T) // 4]
            assert np.isin(heavy, anchors[0, h].cpu().numpy()).all()

    lo, hi = orc.buckets(anchors_to_merge_on(anchors, o_anchors), T)
    o_Kc, o_Vc = orc.merge(Kb, lo, hi), orc.merge(Vb, lo, hi)
    assert_bf16_close(Kc, o_Kc, "merged K")
    assert_bf16_close(Vc, o_Vc, "merged V")

    # the oracle decodes from its own merged rows, rounded to bf16 as the cache stores them
    queue = orc.DecodeQueue(orc.widen_bf16(orc.round_bf16(o_Kc)), orc.widen_bf16(orc.round_bf16(o_Vc)), cap=C + 1)
    cache = ec.ec_cache_init(Kc, Vc, C, C, w.offset)
    ws_d = scratch(ec.ec_decode_workspace(cache))
    out = torch.empty((N, H, D), dtype=torch.bfloat16, device="cuda")
    for s in range(steps):
        qb, kb, vb = (np.ascontiguousarray(x[:, :heads]) for x in wl.decode_step_inputs(w, s, problems))
        want, pos, _ = queue.step(qb, kb, vb, w.scale, policy=orc.POLICY_FIXED, budget=C, offset=w.offset)
        ev, _ = ec.ec_decode_step(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, w.scale, out, ws_d)
        assert ev == (C - w.offset) + (s % w.offset) and pos == C - w.offset
        assert_bf16_close(out, want, f"decode out, step {s}")
    assert cache.len == C


# ---------------------------------------------------------------- retention-ratio policy

@pytest.mark.parametrize("T,ratio,offset,steps,N,H,D", [(200, 0.3, 16, 150, 2, 3, 128), (90, 0.5, 25, 80, 1, 8, 64),
                                                        (64, 1.0, 4, 20, 1, 2, 128)])
def test_decode_ratio_policy_grows_and_evicts_like_the_oracle(T, ratio, offset, steps, N, H, D):
    """The budget follows keep_ratio x tokens seen: some steps append, some evict at the fixed
    truncation location. Same rows must leave on both sides, and outputs must agree."""
    rng = np.random.default_rng(T)
    C = orc.keep_count(T, ratio)
    cap = C + steps
    K0b, V0b = rand_bits(rng, (N, H, C, D)), rand_bits(rng, (N, H, C, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=cap + 1, n_seen=T)
    Kc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    Vc = Guarded((N, H, cap, D), torch.bfloat16, fill=float("nan"))
    Kc.t[:, :, :C] = dev_bf16(K0b)
    Vc.t[:, :, :C] = dev_bf16(V0b)
    cache = ec.ec_cache_init_ratio(Kc.t, Vc.t, C, offset, ratio, T)
    ws = scratch(ec.ec_decode_workspace(cache))
    slot_ids = list(range(C)) + [-1] * (cap - C)
    grew = evicted_n = 0
    for s in range(steps):
        qb, kb, vb = rand_bits(rng, (N, H, D)), rand_bits(rng, (N, H, D)), rand_bits(rng, (N, H, D))
        len_before = cache.len
        want, pos, ident = queue.step(qb, kb, vb, 0.1, policy=orc.POLICY_RATIO, offset=offset, ratio=ratio)
        out = torch.empty((N, H, D), dtype=torch.bfloat16, device="cuda")
        ev, slot = ec.ec_decode_step(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, 0.1, out, ws)
        assert_bf16_close(out, want, f"decode out, step {s}")
        if pos < 0:
            assert ev == -1 and slot == len_before and cache.len == len_before + 1
            grew += 1
        else:
            assert pos == len_before - offset and ev == slot and slot_ids[ev] == ident and cache.len == len_before
            evicted_n += 1
        slot_ids[slot] = queue.next_id - 1
        assert cache.len == queue.len and cache.n_tot == T + s + 1
        assert sorted(slot_ids[:cache.len]) == sorted(queue.identities().tolist())
    assert grew > 0 and (evicted_n > 0 or ratio == 1.0)
    Kc.check("Kc")
    Vc.check("Vc")
    Kdev = host_f64(Kc.t[:, :, :cache.len])
    for j, ident in enumerate(queue.identities().tolist()):
        np.testing.assert_array_equal(Kdev[:, :, slot_ids.index(ident)], queue.K[:, j].reshape(N, H, D))


# ---------------------------------------------------------------- importance from a given normaliser

@pytest.mark.parametrize("N,H,T,D", [(1, 2, 129, 128), (2, 2, 300, 64), (1, 3, 640, 128)])
def test_importance_from_lse_matches_oracle(N, H, T, D):
    rng = np.random.default_rng(T + 11)
    Qb, Kb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    scale = 1.0 / math.sqrt(D)
    want, o_lse = orc.importance(Qb, Kb, scale)
    lse = torch.from_numpy(o_lse.astype(np.float32)).cuda()       # the oracle's normaliser as the input
    scores = Guarded((N, H, T), torch.float32, fill=float("nan"))
    ws = scratch(ec.ec_importance_workspace(N, H, T, D))
    ec.ec_importance_from_lse(dev_bf16(Qb), dev_bf16(Kb), lse, scores.t, scale, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    scores.check("scores")
    assert_rel_close(scores.t, want, SCORE_RTOL, what="scores from lse")


# ---------------------------------------------------------------- ablation variants of the compaction

def gpu_select_compact(Kb, Vb, s32, n_keep, share, protect, compaction):
    N, H, T, D = Kb.shape
    Kc = Guarded((N, H, n_keep, D), torch.bfloat16, fill=float("nan"))
    Vc = Guarded((N, H, n_keep, D), torch.bfloat16, fill=float("nan"))
    anchors = Guarded((N, H, n_keep), torch.int32, fill=-7)
    ws = scratch(ec.ec_select_compact_workspace(N, H, T, D, n_keep, share))
    ec.ec_select_compact(dev_bf16(Kb), dev_bf16(Vb), torch.from_numpy(s32).cuda(), n_keep, share, protect, compaction,
                         Kc.t, Vc.t, anchors.t, None, ws)
    for g, name in ((Kc, "Kc"), (Vc, "Vc"), (anchors, "anchor_pos")):
        g.check(name)
    return Kc.t, Vc.t, anchors.t


@pytest.mark.parametrize("share_kind", ["head", "layer", "sequence"])
@pytest.mark.parametrize("compaction", [ec.EC_COMPACT_MERGE, ec.EC_COMPACT_EVICT])
def test_select_compact_populations_and_eviction(share_kind, compaction):
    B, Lyr, H, T, D, n_keep = 2, 3, 4, 260, 128, 40
    N = B * Lyr
    share = {"head": 1, "layer": H, "sequence": Lyr * H}[share_kind]
    rng = np.random.default_rng(share + compaction)
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    s32 = (rng.random((N, H, T)) ** 3 + 1e-3).astype(np.float32)
    s64 = s32.astype(np.float64).reshape(N * H, T)
    rank = np.repeat(orc.group_mean(s64, share), share, axis=0).reshape(N, H, T)
    want_anchors = orc.select(rank, n_keep, True)
    Kc, Vc, anchors = gpu_select_compact(Kb, Vb, s32, n_keep, share, True, compaction)
    check_anchor_sets(anchors, want_anchors, rank, n_keep, True)
    ga = anchors.cpu().numpy().reshape(N * H // share, share, n_keep)
    assert (ga == ga[:, :1]).all()                               # one anchor set per sharing group
    use = anchors_to_merge_on(anchors, want_anchors)
    if compaction == ec.EC_COMPACT_EVICT:
        np.testing.assert_array_equal(host_f64(Kc), orc.gather(Kb, use))     # copies: bit-exact
        np.testing.assert_array_equal(host_f64(Vc), orc.gather(Vb, use))
    else:
        lo, hi = orc.buckets(use, T)
        assert_bf16_close(Kc, orc.merge(Kb, lo, hi), "merged K")
        assert_bf16_close(Vc, orc.merge(Vb, lo, hi), "merged V")


@pytest.mark.parametrize("N", [20, 64])       # 15 MB per step: successor released after the wait; 47 MB: released at once
def test_decode_steps_overlapped_loop_with_many_units(N):
    """With enough units for one CTA per unit, the native loop lets later steps read the rows no step
    writes (here the first 35 of 45) while earlier steps are still in flight; the ring of the 10 most
    recent rows, which sits in a full block and in the ragged last block, is read after the wait.
    Results must match the one-step calls and the oracle."""
    rng = np.random.default_rng(12)
    H, D, C, d, S = 32, 128, 45, 10, 33
    K0b, V0b = rand_bits(rng, (N, H, C, D)), rand_bits(rng, (N, H, C, D))
    qb, kb, vb = (rand_bits(rng, (S, N, H, D)) for _ in range(3))
    K0, V0 = dev_bf16(K0b), dev_bf16(V0b)
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    Ka, Va, Kb_, Vb_ = K0.clone(), V0.clone(), K0.clone(), V0.clone()
    ca, cb = ec.ec_cache_init(Ka, Va, C, C, d), ec.ec_cache_init(Kb_, Vb_, C, C, d)
    ws = scratch(ec.ec_decode_workspace(ca))
    out_a = torch.empty((S, N, H, D), dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty_like(out_a)
    for s in range(S):
        ec.ec_decode_step(q[s], k[s], v[s], ca, 0.09, out_a[s], ws)
    slots = ec.ec_decode_steps(q, k, v, cb, 0.09, out_b, ws, want_slots=True)
    torch.cuda.synchronize()
    assert slots == [(C - d) + (s % d) for s in range(S)]
    assert torch.equal(Ka, Kb_) and torch.equal(Va, Vb_)
    a, b = host_f64(out_a), host_f64(out_b)
    assert (np.abs(a - b) <= 2.0 ** -7 * np.abs(a) + 1e-6).all()          # same result up to block order
    for (n, h) in [(0, 0), (7, 13), (N - 1, 31)]:
        queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b[n, h][None]), wl.bf16_bits_to_f64(V0b[n, h][None]), cap=C + 1)
        for s in range(S):
            want, _, _ = queue.step(qb[s, n, h][None], kb[s, n, h][None], vb[s, n, h][None], 0.09,
                                    policy=orc.POLICY_FIXED, budget=C, offset=d)
            err = np.abs(b[s, n, h] - want[0])
            assert (err <= 2e-2 + 2.0 ** -8 * np.abs(want[0])).all(), (n, h, s)


# ---------------------------------------------------------------- importance over cache + new instruction

@pytest.mark.parametrize("N,H,Tq,P,D", [(1, 2, 1, 5, 64), (1, 2, 130, 1, 128), (2, 2, 200, 127, 128), (1, 3, 129, 128, 64),
                                        (1, 2, 300, 333, 128), (1, 1, 64, 700, 128), (1, 2, 640, 320, 128)])
def test_importance_prefix_matches_oracle(N, H, Tq, P, D):
    rng = np.random.default_rng(Tq + 3 * P)
    Qb, Kb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, P + Tq, D))
    scale = 1.0 / math.sqrt(D)
    want, want_lse = orc.importance_prefix(Qb, Kb, scale)
    scores = Guarded((N, H, P + Tq), torch.float32, fill=float("nan"))
    lse = Guarded((N, H, Tq), torch.float32, fill=float("nan"))
    ws = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ec.ec_importance_prefix(dev_bf16(Qb), dev_bf16(Kb), scores.t, lse.t, scale, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    scores.check("scores")
    lse.check("lse")
    assert_rel_close(scores.t, want, SCORE_RTOL, what="scores with prefix")
    assert_rel_close(lse.t, want_lse, 1e-3, atol=1e-3, what="lse with prefix")
    np.testing.assert_allclose(host_f64(scores.t).sum(-1), Tq, rtol=1e-3)


# ---------------------------------------------------------------- other importance statistics (Sec. 3.2)

@pytest.mark.parametrize("N,H,Tq,P,D", [(2, 2, 200, 127, 128), (1, 3, 129, 0, 64), (1, 2, 640, 0, 128), (1, 2, 70, 400, 128)])
@pytest.mark.parametrize("stat,beta", [("mean", 0.0), ("max", 0.0), ("moving_average", 0.9), ("moving_average", 0.99)])
def test_importance_statistics_match_oracle(N, H, Tq, P, D, stat, beta):
    rng = np.random.default_rng(7 * Tq + P + len(stat))
    Qb, Kb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, P + Tq, D))
    scale = 1.0 / math.sqrt(D)
    o_stat = {"mean": orc.STAT_MEAN, "max": orc.STAT_MAX, "moving_average": orc.STAT_MOVING_AVERAGE}[stat]
    g_stat = {"mean": ec.EC_STAT_MEAN, "max": ec.EC_STAT_MAX, "moving_average": ec.EC_STAT_MOVING_AVERAGE}[stat]
    want = orc.importance_statistic(Qb, Kb, scale, o_stat, beta)
    _, want_lse = orc.importance_prefix(Qb, Kb, scale)
    scores = Guarded((N, H, P + Tq), torch.float32, fill=float("nan"))
    lse = Guarded((N, H, Tq), torch.float32, fill=float("nan"))
    ws = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ec.ec_importance_statistic(dev_bf16(Qb), dev_bf16(Kb), scores.t, lse.t, scale, g_stat, beta, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    scores.check("scores")
    lse.check("lse")
    assert_rel_close(scores.t, want, SCORE_RTOL, what=f"{stat} importance")
    assert_rel_close(lse.t, want_lse, 1e-3, atol=1e-3, what="lse is the plain one whatever the statistic")


@pytest.mark.parametrize("beta", [0.5, 0.1])
def test_moving_average_long_prompt_small_factor(beta):
    # the exponent of a query's weight reaches -Tq*log2(1/beta) (tens of thousands for the oldest queries); it is
    # counted from the last query, so the newest queries, which carry the weight, keep an exact exponent
    N, H, Tq, D = 1, 2, 4096, 128
    rng = np.random.default_rng(int(beta * 100))
    Qb, Kb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, Tq, D))
    scale = 1.0 / math.sqrt(D)
    want = orc.importance_statistic(Qb, Kb, scale, orc.STAT_MOVING_AVERAGE, beta)
    scores = Guarded((N, H, Tq), torch.float32, fill=float("nan"))
    ws = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ec.ec_importance_statistic(dev_bf16(Qb), dev_bf16(Kb), scores.t, None, scale, ec.EC_STAT_MOVING_AVERAGE, beta, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    scores.check("scores")
    assert_rel_close(scores.t, want, SCORE_RTOL, atol=1e-30, what=f"moving average, beta {beta}")
    np.testing.assert_allclose(host_f64(scores.t).sum(-1), 1.0 - beta ** Tq, rtol=1e-3)


def test_importance_statistic_sum_is_the_prefix_call_and_bad_arguments_are_refused():
    rng = np.random.default_rng(3)
    N, H, Tq, P, D = 1, 2, 150, 20, 128
    Qb, Kb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, P + Tq, D))
    Q, K = dev_bf16(Qb), dev_bf16(Kb)
    a = torch.empty((N, H, P + Tq), dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    ws = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ec.ec_importance_prefix(Q, K, a, None, 0.1, ws)
    ec.ec_importance_statistic(Q, K, b, None, 0.1, ec.EC_STAT_SUM, 0.0, ws)
    assert torch.equal(a, b)
    for stat, beta in [(ec.EC_STAT_MOVING_AVERAGE, 0.0), (ec.EC_STAT_MOVING_AVERAGE, 1.0), (4, 0.5), (-1, 0.5)]:
        with pytest.raises(ec.EcError) as e:
            ec.ec_importance_statistic(Q, K, b, None, 0.1, stat, beta, ws)
        assert e.value.status == ec.EC_ERR_ARG


# ---------------------------------------------------------------- failure path of the bounded waits

def test_bounded_wait_expires_reports_and_leaves_the_context_usable():
    """A barrier that nothing completes: the wait gives up after its limit, the status word says so,
    and the next real call on the same workspace runs normally (no hang, no fault)."""
    rng = np.random.default_rng(2)
    N, H, T, D = 1, 2, 200, 128
    ws = scratch(ec.ec_importance_workspace(N, H, T, D))
    ec.ec_selftest_wait_timeout(ws, 2000)                       # 2 ms
    assert ec.ec_device_status(ws) == 7                         # EC_ERR_TIMEOUT
    assert "timed out" in ec.status_string(7)
    Qb, Kb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    want, _ = orc.importance(Qb, Kb, 0.1)
    scores = torch.empty((N, H, T), dtype=torch.float32, device="cuda")
    ec.ec_importance(dev_bf16(Qb), dev_bf16(Kb), scores, None, 0.1, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK                  # the status word is reset by every call
    assert_rel_close(scores, want, SCORE_RTOL, what="scores after a timed-out self-test")


# ---------------------------------------------------------------- a second instruction on top of the cache

def test_second_instruction_on_top_of_a_decoded_cache():
    """Prompt -> compact -> decode -> a new instruction arrives -> compact [cache ; new rows] -> decode.
    The oracle runs its own chain; the GPU's second stage starts from the oracle's queue (rows placed
    in ring order, as a decoded cache holds them), so both sides see identical inputs."""
    from paper_2407_18121_b200.session import ElasticCacheSession
    rng = np.random.default_rng(99)
    N, H, D, C, d, S1, Tq, S2, scale, ratio = 1, 4, 128, 64, 16, 21, 150, 6, 0.09, 0.5
    # oracle stage 1: a compacted cache of C rows, S1 decode steps
    K0b, V0b = rand_bits(rng, (N, H, C, D)), rand_bits(rng, (N, H, C, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=C + 1)
    for s in range(S1):
        qb, kb, vb = (rand_bits(rng, (N, H, D)) for _ in range(3))
        queue.step(qb, kb, vb, scale, policy=orc.POLICY_FIXED, budget=C, offset=d)
    Kq = orc.round_bf16(queue.K[:, :C].reshape(N, H, C, D))          # queue order, exact (rows are bf16 values)
    Vq = orc.round_bf16(queue.V[:, :C].reshape(N, H, C, D))

    # the same cache as the GPU holds it after S1 evictions: ring rotated by S1 mod d
    sess = ElasticCacheSession(N, H, 2 * C, D, 0.5, d, scale)          # n_keep = C
    assert sess.n_keep == C
    head = S1 % d
    Kp, Vp = np.empty_like(Kq), np.empty_like(Vq)
    for pos in range(C):
        slot = pos if pos < C - d else C - d + (head + (pos - (C - d))) % d
        Kp[:, :, slot], Vp[:, :, slot] = Kq[:, :, pos], Vq[:, :, pos]
    sess.Kc[:, :, :C] = dev_bf16(Kp)
    sess.Vc[:, :, :C] = dev_bf16(Vp)
    sess.cache = ec.ec_cache_init(sess.Kc, sess.Vc, C, C, d)
    sess.cache.ring_head = head
    order = sess.logical_slots()
    np.testing.assert_array_equal(host_bits(sess.Kc[:, :, order]), Kq)    # queue order recovered

    # the new instruction
    Qn, Kn, Vn = (rand_bits(rng, (N, H, Tq, D)) for _ in range(3))
    K_all, V_all = np.concatenate([Kq, Kn], 2), np.concatenate([Vq, Vn], 2)
    o_scores, _ = orc.importance_prefix(Qn, K_all, scale)
    C2 = orc.keep_count(C + Tq, ratio)
    o_anch = orc.select(o_scores, C2, True)
    nxt = sess.recompress(dev_bf16(Qn), dev_bf16(Kn), dev_bf16(Vn), ratio)
    assert nxt.n_keep == C2
    assert_rel_close(nxt.scores, o_scores, SCORE_RTOL, what="scores over cache + new instruction")
    check_anchor_sets(nxt.anchor_pos, o_anch, o_scores, C2, True)
    lo, hi = orc.buckets(anchors_to_merge_on(nxt.anchor_pos, o_anch), C + Tq)
    o_K, o_V = orc.merge(K_all, lo, hi), orc.merge(V_all, lo, hi)
    assert_bf16_close(nxt.Kc, o_K, "re-merged K")
    assert_bf16_close(nxt.Vc, o_V, "re-merged V")

    queue2 = orc.DecodeQueue(orc.widen_bf16(orc.round_bf16(o_K)), orc.widen_bf16(orc.round_bf16(o_V)), cap=C2 + 1)
    out = torch.empty((N, H, D), dtype=torch.bfloat16, device="cuda")
    for s in range(S2):
        qb, kb, vb = (rand_bits(rng, (N, H, D)) for _ in range(3))
        want, _, _ = queue2.step(qb, kb, vb, scale, policy=orc.POLICY_FIXED, budget=C2, offset=d)
        ec.ec_decode_step(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), nxt.cache, scale, out, nxt.ws_dec)
        assert_bf16_close(out, want, f"decode after the second instruction, step {s}")


@pytest.mark.parametrize("N,H,D,C,len0,offset,steps,Tq", [
    (2, 3, 128, 40, 40, 16, 23, 50),      # full cache, ring rotated by 23 mod 16
    (1, 5, 64, 33, 33, 7, 14, 1),         # whole turns of the ring (14 = 2 * 7), one new row
    (1, 4, 128, 48, 20, 16, 11, 30),      # still below its budget: no ring yet
    (2, 2, 64, 24, 10, 23, 40, 9),        # grows to the budget, then evicts; offset = budget - 1
])
def test_cache_concat_restores_queue_order(N, H, D, C, len0, offset, steps, Tq):
    """ec_cache_concat after a decode chain: the oracle's queue (oldest first), then the new rows, bit for bit."""
    rng = np.random.default_rng(1000 + C + steps)
    scale = 1.0 / math.sqrt(D)
    K0b, V0b = rand_bits(rng, (N, H, len0, D)), rand_bits(rng, (N, H, len0, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=C + 1)
    Kc = torch.zeros((N, H, C, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    Kc[:, :, :len0], Vc[:, :, :len0] = dev_bf16(K0b), dev_bf16(V0b)
    cache = ec.ec_cache_init(Kc, Vc, len0, C, offset)
    ws = scratch(ec.ec_decode_workspace(cache))
    qb, kb, vb = (rand_bits(rng, (steps, N, H, D)) for _ in range(3))
    for s in range(steps):
        queue.step(qb[s], kb[s], vb[s], scale, policy=orc.POLICY_FIXED, budget=C, offset=offset)
    out = torch.empty((steps, N, H, D), dtype=torch.bfloat16, device="cuda")
    ec.ec_decode_steps(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, scale, out, ws)
    P = cache.len
    assert P == queue.len == min(C, len0 + steps)
    Knb, Vnb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, Tq, D))
    K_all = Guarded((N, H, P + Tq, D), torch.bfloat16, fill=float("nan"))
    V_all = Guarded((N, H, P + Tq, D), torch.bfloat16, fill=float("nan"))
    ec.ec_cache_concat(cache, dev_bf16(Knb), dev_bf16(Vnb), K_all.t, V_all.t)
    K_all.check("K_all")
    V_all.check("V_all")
    want_K = np.concatenate([orc.round_bf16(queue.K[:, :P].reshape(N, H, P, D)), Knb], 2)
    want_V = np.concatenate([orc.round_bf16(queue.V[:, :P].reshape(N, H, P, D)), Vnb], 2)
    np.testing.assert_array_equal(host_bits(K_all.t), want_K)
    np.testing.assert_array_equal(host_bits(V_all.t), want_V)


@pytest.mark.parametrize("N,H,D,T,ratio,offset,steps,Tq", [
    (2, 3, 128, 60, 0.5, 8, 45, 17),      # alternates between growing and evicting
    (1, 4, 64, 100, 0.3, 25, 90, 40),     # the paper's recent distance; mostly evicts
    (1, 2, 128, 40, 1.0, 4, 30, 5),       # ratio 1: never evicts, slots stay in order
    (1, 2, 64, 3000, 0.4, 16, 700, 3),    # more rows than one slot list per launch holds (896)
])
def test_cache_concat_on_a_retention_ratio_cache(N, H, D, T, ratio, offset, steps, Tq):
    """Sec. 3.1 (the instruction stage takes in the chat history) on top of Sec. 3.3's literal generation
    rule: after a chain of grow / evict steps the physical slots are in no simple order; the tracked
    queue order must reproduce the oracle's queue, oldest first, bit for bit, followed by the new rows."""
    rng = np.random.default_rng(T + steps)
    scale = 1.0 / math.sqrt(D)
    len0 = orc.keep_count(T, ratio)
    cap = len0 + steps
    K0b, V0b = rand_bits(rng, (N, H, len0, D)), rand_bits(rng, (N, H, len0, D))
    queue = orc.DecodeQueue(wl.bf16_bits_to_f64(K0b), wl.bf16_bits_to_f64(V0b), cap=cap + 1, n_seen=T)
    Kc = torch.zeros((N, H, cap, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    Kc[:, :, :len0], Vc[:, :, :len0] = dev_bf16(K0b), dev_bf16(V0b)
    cache = ec.ec_cache_init_ratio(Kc, Vc, len0, offset, ratio, T)
    ws = scratch(ec.ec_decode_workspace(cache))
    qb, kb, vb = (rand_bits(rng, (steps, N, H, D)) for _ in range(3))
    for s in range(steps):
        queue.step(qb[s], kb[s], vb[s], scale, policy=orc.POLICY_RATIO, offset=offset, ratio=ratio)
    out = torch.empty((steps, N, H, D), dtype=torch.bfloat16, device="cuda")
    ec.ec_decode_steps(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), cache, scale, out, ws)
    P = cache.len
    assert P == queue.len
    order = [cache.queue_slots_host[j] for j in range(P)]
    assert sorted(order) == list(range(P)) if ratio == 1.0 else len(set(order)) == P
    Knb, Vnb = rand_bits(rng, (N, H, Tq, D)), rand_bits(rng, (N, H, Tq, D))
    K_all = Guarded((N, H, P + Tq, D), torch.bfloat16, fill=float("nan"))
    V_all = Guarded((N, H, P + Tq, D), torch.bfloat16, fill=float("nan"))
    ec.ec_cache_concat(cache, dev_bf16(Knb), dev_bf16(Vnb), K_all.t, V_all.t)
    K_all.check("K_all")
    V_all.check("V_all")
    want_K = np.concatenate([orc.round_bf16(queue.K[:, :P].reshape(N, H, P, D)), Knb], 2)
    want_V = np.concatenate([orc.round_bf16(queue.V[:, :P].reshape(N, H, P, D)), Vnb], 2)
    np.testing.assert_array_equal(host_bits(K_all.t), want_K)
    np.testing.assert_array_equal(host_bits(V_all.t), want_V)
    # the history feeds the importance of the new instruction exactly as a fixed-budget cache's does
    Qnb = rand_bits(rng, (N, H, Tq, D))
    scores = torch.empty((N, H, P + Tq), dtype=torch.float32, device="cuda")
    ws_i = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ec.ec_importance_prefix(dev_bf16(Qnb), K_all.t, scores, None, scale, ws_i)
    assert ec.ec_device_status(ws_i) == ec.EC_OK
    o_scores, _ = orc.importance_prefix(Qnb, want_K, scale)
    assert_rel_close(scores, o_scores, SCORE_RTOL, what="importance over the ratio cache's history")


def test_cache_concat_rejects_an_untracked_ratio_cache_and_bad_shapes():
    N, H, D, C = 1, 2, 64, 16
    Kc = torch.zeros((N, H, C + 8, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    new = torch.zeros((N, H, 4, D), dtype=torch.bfloat16, device="cuda")
    all_ = torch.zeros((N, H, C + 4, D), dtype=torch.bfloat16, device="cuda")
    ratio_cache = ec.ec_cache_init_ratio(Kc, Vc, C, 4, 0.5, 32, track_order=False)
    with pytest.raises(ec.EcError) as e:
        ec.ec_cache_concat(ratio_cache, new, new, all_, all_.clone())
    assert e.value.status == ec.EC_ERR_ARG
    fixed = ec.ec_cache_init(Kc, Vc, C, C, 4)
    with pytest.raises(ValueError):
        ec.ec_cache_concat(fixed, new, new, all_[:, :, :-1].contiguous(), all_[:, :, :-1].contiguous())


# ---------------------------------------------------------------- host-resident tensors

def test_host_entry_points_match_the_device_path():
    """ec_compress_host / ec_decode_steps_host only add copies: same anchors, cache and outputs as the
    device-resident calls, including a step count that does not divide into whole chunks."""
    from paper_2407_18121_b200.session import ElasticCacheSession
    w = wl.WORKLOADS["tiny"]
    Qb, Kb, Vb = wl.prompt(w)
    S = 23
    qb, kb, vb = wl.decode_inputs(w, S)
    N, H, T, D = Qb.shape

    def pinned(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).pin_memory()

    a = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    a.compress(dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb))
    out_a = torch.empty((S, N, H, D), dtype=torch.bfloat16, device="cuda")
    a.decode(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), out_a)

    b = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    anchors_h = torch.full((N, H, b.n_keep), -1, dtype=torch.int32).pin_memory()
    out_h = torch.zeros((S, N, H, D), dtype=torch.bfloat16).pin_memory()
    b.compress_host(pinned(Qb), pinned(Kb), pinned(Vb), anchors_h)
    b.decode_host(pinned(qb), pinned(kb), pinned(vb), out_h, chunk=5)
    torch.cuda.synchronize()
    assert torch.equal(a.anchor_pos.cpu(), anchors_h)
    assert torch.equal(a.Kc, b.Kc) and torch.equal(a.Vc, b.Vc)
    assert torch.equal(out_a.cpu(), out_h)
    assert (b.cache.len, b.cache.ring_head, b.cache.step) == (a.cache.len, a.cache.ring_head, a.cache.step)


# ---------------------------------------------------------------- CUDA graph capture of a whole pass

def test_whole_pass_can_be_captured_in_a_cuda_graph_and_replayed():
    """Every call only enqueues work on the given stream, so a pass (importance, select/merge, decode
    loop) can be recorded once and replayed. The host-side cache bookkeeping is replayed implicitly:
    the pass starts from compress(), so each replay sees the same slot sequence."""
    from paper_2407_18121_b200.session import ElasticCacheSession
    w = wl.WORKLOADS["tiny"]
    Qb, Kb, Vb = wl.prompt(w)
    S = 12
    qb, kb, vb = wl.decode_inputs(w, S)
    N, H, T, D = Qb.shape
    Q, K, V = dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)
    q, k, v = dev_bf16(qb), dev_bf16(kb), dev_bf16(vb)
    sess = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    out_eager = torch.empty((S, N, H, D), dtype=torch.bfloat16, device="cuda")
    sess.compress(Q, K, V)                                   # eager reference (also warms everything up)
    sess.decode(q, k, v, out_eager)
    torch.cuda.synchronize()
    Kc_ref, anchors_ref = sess.Kc.clone(), sess.anchor_pos.clone()

    out_graph = torch.zeros_like(out_eager)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            sess.compress(Q, K, V)
            sess.decode(q, k, v, out_graph)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        out_graph.zero_()
        sess.Kc.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out_graph, out_eager)
        assert torch.equal(sess.Kc, Kc_ref) and torch.equal(sess.anchor_pos, anchors_ref)
    assert ec.ec_device_status(sess.ws_imp) == ec.EC_OK


def test_ratio_policy_through_the_overlapped_native_loop():
    """Growing cache + native loop with one CTA per unit: the row the previous step appended (or
    overwrote) is the one read late. Must equal the one-step calls."""
    rng = np.random.default_rng(31)
    N, H, D, C, d, S, T, ratio = 20, 32, 128, 41, 9, 30, 100, 0.41
    cap = C + S
    K0, V0 = (dev_bf16(rand_bits(rng, (N, H, cap, D))) for _ in range(2))
    q, k, v = (dev_bf16(rand_bits(rng, (S, N, H, D))) for _ in range(3))
    Ka, Va, Kb_, Vb_ = K0.clone(), V0.clone(), K0.clone(), V0.clone()
    ca = ec.ec_cache_init_ratio(Ka, Va, C, d, ratio, T)
    cb = ec.ec_cache_init_ratio(Kb_, Vb_, C, d, ratio, T)
    ws = scratch(ec.ec_decode_workspace(ca))
    out_a = torch.empty((S, N, H, D), dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty_like(out_a)
    slots_a = [ec.ec_decode_step(q[s], k[s], v[s], ca, 0.09, out_a[s], ws)[0] for s in range(S)]
    slots_b = ec.ec_decode_steps(q, k, v, cb, 0.09, out_b, ws, want_slots=True)
    torch.cuda.synchronize()
    assert slots_a == slots_b and -1 in slots_a and any(x >= 0 for x in slots_a)    # grew and evicted
    assert (ca.len, ca.n_tot, ca.recent_head) == (cb.len, cb.n_tot, cb.recent_head)
    assert torch.equal(Ka[:, :, :ca.len], Kb_[:, :, :cb.len]) and torch.equal(Va[:, :, :ca.len], Vb_[:, :, :cb.len])
    a, b = host_f64(out_a), host_f64(out_b)
    assert (np.abs(a - b) <= 2.0 ** -7 * np.abs(a) + 1e-6).all()


# ---------------------------------------------------------------- seeded random shapes

def test_random_shapes_select_merge_and_decode():
    """Forty seeded shapes off the beaten path (prompt lengths around warp / tile / slice borders,
    keep counts from 1 to T, both head sizes, shared populations, long offsets)."""
    rng = np.random.default_rng(20240718)
    for case in range(40):
        D = int(rng.choice([64, 128]))
        H = int(rng.integers(1, 5))
        N = int(rng.integers(1, 4))
        T = int(rng.choice([1, 2, 3, 31, 32, 33, 63, 255, 256, 257, 511, 513, 1023, 1024, 1025, 1500, 2049]))
        n_keep = int(rng.integers(1, T + 1))
        protect = bool(rng.integers(0, 2))
        share = int(rng.choice([1, H]))
        Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
        levels = int(rng.choice([3, 50, 100000]))                      # few levels -> many exact ties
        s32 = (rng.integers(1, levels + 1, size=(N, H, T)) / levels).astype(np.float32)
        rank = np.repeat(orc.group_mean(s32.astype(np.float64).reshape(N * H, T), share), share, 0).reshape(N, H, T)
        want = orc.select(rank, n_keep, protect)
        Kc, Vc, anchors = gpu_select_compact(Kb, Vb, s32, n_keep, share, protect, ec.EC_COMPACT_MERGE)
        exact, total = check_anchor_sets(anchors, want, rank, n_keep, protect)
        if share == 1:
            assert exact == total, (case, N, H, T, D, n_keep, protect)
        lo, hi = orc.buckets(anchors_to_merge_on(anchors, want), T)
        assert_bf16_close(Kc, orc.merge(Kb, lo, hi), f"merged K, case {case}")
        assert_bf16_close(Vc, orc.merge(Vb, lo, hi), f"merged V, case {case}")
    for case in range(12):
        D = int(rng.choice([64, 128]))
        N, H = int(rng.integers(1, 30)), int(rng.integers(1, 33))
        C = int(rng.integers(2, 150))
        offset = int(rng.integers(1, C))
        len0 = int(rng.integers(0, C + 1))
        run_decode_case(N, H, D, C, C + int(rng.integers(0, 5)), len0, offset, int(rng.integers(1, 12)),
                        float(rng.uniform(0.05, 0.3)), seed=1000 + case)
