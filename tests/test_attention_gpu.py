"""GPU parity of ec_prefill_attention (causal attention of the prompt tokens with the row
normaliser, and the importance of Eq. 1 from the column-sum pass alone) against the CPU oracle."""
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
    return wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * sigma)


def run_attention(Qb, Kb, Vb, scale, want_scores=True):
    N, H, Tq, D = Qb.shape
    Tk = Kb.shape[2]
    out = Guarded((N, H, Tq, D), torch.bfloat16, fill=float("nan"))
    lse = Guarded((N, H, Tq), torch.float32, fill=float("nan"))
    scores = Guarded((N, H, Tk), torch.float32, fill=float("nan")) if want_scores else None
    ws = scratch(ec.ec_importance_workspace(N, H, Tq, D))
    ws.fill_(0xA5)                                                  # a dirty workspace must not matter
    ec.ec_prefill_attention(dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb), out.t, lse.t, scores.t if scores else None, scale, ws)
    assert ec.ec_device_status(ws) == ec.EC_OK
    out.check("out")
    lse.check("lse")
    if scores:
        scores.check("scores")
    return out.t, lse.t, scores.t if scores else None


# one tile, ragged tiles, several tiles with a ragged tail, both head dimensions, with and without a prefix
SHAPES = [(1, 1, 1, 0, 128), (2, 2, 100, 0, 128), (1, 2, 128, 0, 128), (1, 3, 129, 0, 64), (2, 2, 300, 0, 128),
          (1, 4, 640, 0, 128), (1, 2, 515, 0, 64), (2, 2, 200, 127, 128), (1, 2, 70, 400, 128), (1, 2, 33, 256, 64),
          (1, 1, 1, 300, 128)]


@pytest.mark.parametrize("N,H,Tq,P,D", SHAPES)
def test_prefill_attention_matches_oracle(N, H, Tq, P, D):
    rng = np.random.default_rng(1000 * Tq + P + D)
    Qb = rand_bits(rng, (N, H, Tq, D))
    Kb, Vb = rand_bits(rng, (N, H, P + Tq, D)), rand_bits(rng, (N, H, P + Tq, D))
    scale = 1.0 / math.sqrt(D)
    want_out, want_lse = orc.attention_prefix(Qb, Kb, Vb, scale)
    want_scores, _ = orc.importance_prefix(Qb, Kb, scale)
    out, lse, scores = run_attention(Qb, Kb, Vb, scale)
    assert_bf16_close(out, want_out, "attention output")
    assert_rel_close(lse, want_lse, 1e-3, atol=1e-3, what="lse")
    assert_rel_close(scores, want_scores, SCORE_RTOL, what="scores from the attention kernel's normaliser")
    np.testing.assert_allclose(host_f64(scores).sum(-1), Tq, rtol=1e-3)
    # run to run identical
    out2, lse2, scores2 = run_attention(Qb, Kb, Vb, scale)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    assert torch.equal(lse, lse2) and torch.equal(scores, scores2)


def test_prefill_attention_peaked_rows_raise_the_running_maximum():
    # logits that grow towards the early keys, which a query tile meets last (its key tiles run from the
    # diagonal down to tile 0): the running maximum is raised, and the accumulator rescaled, several times
    N, H, T, D = 1, 2, 520, 128
    rng = np.random.default_rng(5)
    Q = rng.standard_normal((N, H, T, D)).astype(np.float32)
    K = rng.standard_normal((N, H, T, D)).astype(np.float32)
    u = rng.standard_normal(D).astype(np.float32)
    u /= np.linalg.norm(u)
    Q += 6.0 * u
    K += (np.linspace(4.0, 0.0, T, dtype=np.float32)[None, None, :, None] ** 2) * u
    Qb, Kb = wl.to_bf16_bits(Q), wl.to_bf16_bits(K)
    Vb = rand_bits(rng, (N, H, T, D))
    scale = 1.0
    want_out, want_lse = orc.attention_prefix(Qb, Kb, Vb, scale)
    want_scores, _ = orc.importance_prefix(Qb, Kb, scale)
    out, lse, scores = run_attention(Qb, Kb, Vb, scale)
    assert_bf16_close(out, want_out, "attention output (peaked)")
    assert_rel_close(lse, want_lse, 1e-3, atol=1e-3, what="lse (peaked)")
    assert_rel_close(scores, want_scores, SCORE_RTOL, atol=1e-30, what="scores (peaked)")


def test_prefill_attention_special_values():
    N, H, T, D = 1, 2, 260, 128
    rng = np.random.default_rng(9)
    Kb, Vb = rand_bits(rng, (N, H, T, D)), rand_bits(rng, (N, H, T, D))
    # zero queries: every row is the running mean of the values
    Qb = wl.to_bf16_bits(np.zeros((N, H, T, D), np.float32))
    out, lse, _ = run_attention(Qb, Kb, Vb, 0.3, want_scores=False)
    v = wl.bf16_bits_to_f64(Vb)
    want = np.cumsum(v, 2) / np.arange(1, T + 1)[None, None, :, None]
    assert_bf16_close(out, want, "running mean")
    assert_rel_close(lse, np.broadcast_to(np.log(np.arange(1, T + 1)), (N, H, T)), 1e-3, atol=1e-3, what="lse = log(m+1)")
    # constant values come out unchanged
    Qb = rand_bits(rng, (N, H, T, D))
    const = wl.to_bf16_bits(np.broadcast_to(np.linspace(-3, 3, D, dtype=np.float32), (N, H, T, D)).copy())
    out, _, _ = run_attention(Qb, Kb, const, 1.0 / math.sqrt(D), want_scores=False)
    assert_bf16_close(out, wl.bf16_bits_to_f64(const), "constant values")


def test_prefill_attention_refuses_bad_arguments():
    N, H, T, D = 1, 1, 64, 128
    Q = torch.zeros(N, H, T, D, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(Q)
    ws = scratch(ec.ec_importance_workspace(N, H, T, D))
    with pytest.raises(ec.EcError) as e:
        ec.ec_prefill_attention(Q, Q, Q, out, None, None, -1.0, ws)
    assert e.value.status == ec.EC_ERR_ARG
    with pytest.raises(ec.EcError) as e:
        ec.ec_prefill_attention(Q, Q, Q, out, None, None, 1.0, ws[:128])
    assert e.value.status == ec.EC_ERR_WORKSPACE


def _check_sampled_rows(w, problems, units, row_blocks):
    """The whole batch of `problems` on the GPU in one call; the oracle on sampled row blocks of sampled units
    (a block of query rows m0..m1 of a unit is the prefix form with P = m0 earlier keys: the same rows)."""
    Qb, Kb, Vb = wl.prompt(w, problems)
    N, H, T, D = Qb.shape
    out, lse, scores = run_attention(Qb, Kb, Vb, w.scale)
    out_h, lse_h, scores_h = host_f64(out), host_f64(lse), host_f64(scores)
    assert np.isfinite(out_h).all()
    np.testing.assert_allclose(scores_h.sum(-1), T, rtol=1e-3)
    for (n, h) in units:
        for (m0, m1) in row_blocks:
            want_out, want_lse = orc.attention_prefix(Qb[n, h, m0:m1][None], Kb[n, h, :m1][None], Vb[n, h, :m1][None], w.scale)
            err = np.abs(out_h[n, h, m0:m1] - want_out[0])
            assert (err <= 2e-2 + 2.0 ** -8 * np.abs(want_out[0])).all(), (n, h, m0, float(err.max()))
            np.testing.assert_allclose(lse_h[n, h, m0:m1], want_lse[0], rtol=1e-3, atol=1e-3)
    # the scores are the ones the two-pass call gives (same kernels for the column sums, another normaliser)
    Q, K = dev_bf16(Qb), dev_bf16(Kb)
    ref = torch.empty_like(scores)
    ws = scratch(ec.ec_importance_workspace(N, H, T, D))
    ec.ec_importance(Q, K, ref, None, w.scale, ws)
    torch.testing.assert_close(scores, ref, rtol=2e-4, atol=0)


def test_prefill_attention_7b_batch8_shapes_full_length():
    # 1024-token prompts of the batch-8 7B configuration, 8 problems = 256 units in one launch
    w = wl.WORKLOADS["llava7b_b8"]
    _check_sampled_rows(w, list(range(8)), [(0, 0), (3, 17), (7, 31)], [(0, 130), (500, 640), (896, 1024)])


def test_prefill_attention_long_context_units_full_length():
    # 8192-token units of the long-context configuration (64 key tiles per query tile at the end)
    w = wl.WORKLOADS["long8k"]
    _check_sampled_rows(w, [0, 1], [(0, 0), (1, 31)], [(0, 129), (4000, 4100), (8064, 8192)])


def test_session_compress_with_attention_gives_the_same_cache():
    # the prompt call through the attention kernel: the anchors and the merged cache are those of the
    # two-pass call wherever the scores do not tie at the threshold (they agree to a few fp32 ulps)
    from paper_2407_18121_b200.session import ElasticCacheSession
    w = wl.WORKLOADS["tiny"]
    Qb, Kb, Vb = wl.prompt(w)
    N, H, T, D = Qb.shape
    Q, K, V = dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)
    a = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    b = ElasticCacheSession(N, H, T, D, w.keep_ratio, w.offset, w.scale)
    a.compress(Q, K, V)
    out = torch.empty_like(Q)
    b.compress_with_attention(Q, K, V, out)
    assert ec.ec_device_status(b.ws_imp) == ec.EC_OK
    want_out, _ = orc.attention_prefix(Qb, Kb, Vb, w.scale)
    assert_bf16_close(out, want_out, "attention output through the session")
    torch.testing.assert_close(b.scores, a.scores, rtol=2e-4, atol=0)
    same = (a.anchor_pos == b.anchor_pos).all(dim=-1)
    assert same.float().mean().item() >= 0.75
    assert torch.equal(a.Kc[same].view(torch.int16), b.Kc[same].view(torch.int16))
    assert torch.equal(a.Vc[same].view(torch.int16), b.Vc[same].view(torch.int16))
    assert b.cache.len == b.n_keep
