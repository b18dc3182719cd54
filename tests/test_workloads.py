"""The seeded input generators: shapes, determinism and the structure each recipe promises."""
import numpy as np

from paper_2407_18121_b200 import workloads as wl


def test_shapes_and_determinism():
    w = wl.WORKLOADS["tiny"]
    Q, K, V = wl.prompt(w)
    assert Q.shape == K.shape == V.shape == (1, 8, 256, 64) and Q.dtype == np.uint16
    Q2, K2, V2 = wl.prompt(w)
    assert (Q == Q2).all() and (K == K2).all() and (V == V2).all()
    q, k, v = wl.decode_inputs(w)
    assert q.shape == (32, 1, 8, 64)
    q1, _, _ = wl.decode_step_inputs(w, 5)
    assert (q[5] == q1).all()


def test_problem_subset_matches_full_draw():
    w = wl.WORKLOADS["llava7b_b1"].shrunk(layers=32)
    Qs, Ks, Vs = wl.prompt(w, problems=[3, 17])
    Q3, K3, V3 = wl.prompt_problem(w, 3)
    assert (Qs[0] == Q3).all() and (Ks[0] == K3).all() and (Vs[0] == V3).all()
    qa, _, _ = wl.decode_step_inputs(w, 2)
    qb, _, _ = wl.decode_step_inputs(w, 2, problems=[3, 17])
    assert (qa[[3, 17]] == qb).all()


def test_peaked_recipe_has_four_heavy_keys_per_head():
    w = wl.WORKLOADS["tiny"]
    _, K, _ = wl.prompt(w)
    k = wl.bf16_bits_to_f64(K)[0]
    norms = np.linalg.norm(k, axis=-1)            # [H, T]
    for h in range(w.heads):
        top = np.sort(norms[h])[::-1]
        assert top[3] > 2.0 and top[4] < 2.0      # boosted rows have norm ~3, the rest ~1


def test_lowrank_recipe_makes_image_tokens_redundant():
    w = wl.WORKLOADS["llava7b_b1"]
    _, K, V = wl.prompt_problem(w, 0)
    k = wl.bf16_bits_to_f64(K)[0]                 # head 0: [T, D]
    img, txt = k[: w.n_image], k[w.n_image:]
    assert abs(txt.var() - 1.0) < 0.1
    assert abs(img.var() - 5.0) < 0.6             # 1 + rank * (2/sqrt(rank))^2 = 5
    sv = np.linalg.svd(img - img.mean(0), compute_uv=False)
    assert sv[w.rank - 1] > 1.5 * sv[w.rank]      # a rank-8 component above the noise floor


def test_zipf_recipe_is_heavy_tailed():
    w = wl.WORKLOADS["long8k"].shrunk(batch=1, layers=1)
    w = type(w)(**{**w.__dict__, "heads": 1, "prompt_len": 512})
    Q, K, _ = wl.prompt_problem(w, 0)
    q, k = wl.bf16_bits_to_f64(Q)[0], wl.bf16_bits_to_f64(K)[0]
    proj = k @ q.mean(0) / np.linalg.norm(q.mean(0))
    s = np.sort(proj)[::-1]
    assert s[0] > 4.0 and s[0] > 2.0 * s[4]       # the rank-1 position stands far above the rest
