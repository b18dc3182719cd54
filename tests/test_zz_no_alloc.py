"""ec_decode_step_noalloc — the decode step for hosts that may not allocate device memory
(memory pools that own the whole GPU, plug-in hooks, latency-critical loops) — must give what
ec_decode_step gives. Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from paper_2407_18121_b200 import binding as ec
from paper_2407_18121_b200 import workloads as wl
from helpers import BF16_ATOL, BF16_RTOL, dev_bf16, host_f64, scratch

pytestmark = pytest.mark.gpu


def rand_bits(rng, shape):
    return wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


@pytest.mark.parametrize("N,H,D,C,offset", [(1, 8, 64, 600, 16),      # few units: rows split over three CTAs, scratch in use
                                            (2, 4, 128, 130, 25)])
def test_noalloc_matches_workspace_version_twice_in_a_row(N, H, D, C, offset):
    rng = np.random.default_rng(C)
    K0, V0 = dev_bf16(rand_bits(rng, (N, H, C, D))), dev_bf16(rand_bits(rng, (N, H, C, D)))
    Ka, Va, Kb, Vb = K0.clone(), V0.clone(), K0.clone(), V0.clone()
    ca, cb = ec.ec_cache_init(Ka, Va, C, C, offset), ec.ec_cache_init(Kb, Vb, C, C, offset)
    ws = scratch(ec.ec_decode_workspace(ca))
    assert ec.ec_decode_workspace(cb) <= ec.ec_decode_noalloc_capacity()
    for step in range(2):                                   # two calls in a row share the built-in scratch
        q, k, v = (dev_bf16(rand_bits(rng, (N, H, D))) for _ in range(3))
        out_a = torch.full((N, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        out_b = torch.full_like(out_a, float("nan"))
        ev_a, slot_a = ec.ec_decode_step(q, k, v, ca, 0.125, out_a, ws)
        ev_b, slot_b = ec.ec_decode_step_noalloc(q, k, v, cb, 0.125, out_b)
        torch.cuda.synchronize()
        assert (ev_a, slot_a) == (ev_b, slot_b) == (C - offset + step, C - offset + step)
        want, got = host_f64(out_a), host_f64(out_b)
        assert np.isfinite(got).all()
        assert (np.abs(got - want) <= BF16_ATOL + BF16_RTOL * np.abs(want)).all()
        assert torch.equal(Ka, Kb) and torch.equal(Va, Vb)  # the new row went to the same slot
    assert (cb.len, cb.ring_head, cb.step) == (ca.len, ca.ring_head, ca.step)


def test_noalloc_rejects_a_cache_beyond_its_capacity():
    N, H, D, C = 64, 128, 128, 4            # 8192 units: the workspace rule asks for more than 2 MiB
    Kc = torch.zeros((N, H, C, D), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    cache = ec.ec_cache_init(Kc, Vc, C, C, 1)
    assert ec.ec_decode_workspace(cache) > ec.ec_decode_noalloc_capacity()
    x = torch.zeros((N, H, D), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(x)
    with pytest.raises(ec.EcError) as err:
        ec.ec_decode_step_noalloc(x, x, x, cache, 1.0, out)
    assert err.value.status == 8 and "too large" in str(err.value)
    assert (cache.len, cache.step) == (C, 0)
