"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
declared symbol, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from oracle import ec_oracle as orc
from paper_2407_18121_b200 import binding as ec
from paper_2407_18121_b200 import build as ecbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    ecbuild.build()
    return ec.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "ec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ec_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert len(names) >= 11
    for n in names:
        assert hasattr(L, n), f"{n} declared in ec.h but not exported"
    assert sorted(ec.EXPORTS) == names


def test_keep_count_matches_oracle_rule(L):
    for T in (1, 2, 7, 100, 256, 640, 1024, 2048, 8192, 16384):
        for r in (0.0, 0.05, 0.1, 0.2, 0.25, 0.3, 0.5, 0.7, 0.75, 0.9, 1.0):
            assert ec.ec_keep_count(T, r) == orc.keep_count(T, r), (T, r)
    assert ec.ec_keep_count(0, 0.5) == 0 and ec.ec_keep_count(10, 1.5) == 0


def test_status_strings(L):
    seen = {ec.status_string(s) for s in range(8)}
    assert len(seen) == 8 and ec.status_string(99) == "unknown status"


def test_importance_rejects_bad_arguments_on_the_host(L):
    p = 0x10000  # fake, aligned, never dereferenced: every case below fails validation first
    f = L.ec_importance
    assert f(None, p, p, None, 1, 1, 16, 64, 1.0, p, 1 << 20, None) == 1          # NULL
    assert f(p, p, p, None, 1, 1, 16, 96, 1.0, p, 1 << 20, None) == 2             # D
    assert f(p, p, p, None, 1, 1, 0, 64, 1.0, p, 1 << 20, None) == 2              # T
    assert f(p + 2, p, p, None, 1, 1, 16, 64, 1.0, p, 1 << 20, None) == 3         # alignment
    assert f(p, p, p, None, 1, 1, 16, 64, -1.0, p, 1 << 20, None) == 4            # scale
    assert f(p, p, p, None, 1, 1, 16, 64, 1.0, None, 0, None) == 5                # workspace
    assert f(p, p, p, None, 1, 1, 16, 64, 1.0, p, 16, None) == 5
    assert L.ec_importance_workspace(1, 1, 16, 64) >= 256 + 64
    assert L.ec_importance_workspace(1, 1, 16, 100) == 0


def test_select_merge_rejects_bad_arguments_on_the_host(L):
    p = 0x10000
    f = L.ec_select_merge
    ok_ws = 1 << 20
    assert f(p, p, None, 1, 1, 16, 64, 8, 0, 0, p, p, 8, p, None, p, ok_ws, None) == 1
    assert f(p, p, p, 1, 1, 16, 64, 0, 0, 0, p, p, 8, p, None, p, ok_ws, None) == 4    # n_keep
    assert f(p, p, p, 1, 1, 16, 64, 17, 0, 0, p, p, 32, p, None, p, ok_ws, None) == 4
    assert f(p, p, p, 1, 1, 16, 64, 8, 0, 0, p, p, 7, p, None, p, ok_ws, None) == 4    # cap < n_keep
    assert f(p, p, p, 1, 1, 16, 64, 8, 2, 0, p, p, 8, p, None, p, ok_ws, None) == 4    # population
    assert f(p, p, p, 1, 1, 16, 64, 8, 0, 0, p + 8, p, 8, p, None, p, ok_ws, None) == 3
    assert f(p, p, p, 1, 1, 16, 64, 8, 0, 0, p, p, 8, p, None, None, 0, None) == 5


def test_cache_init_and_decode_validation(L):
    p = 0x10000
    c = ec.ec_cache()
    init = L.ec_cache_init
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 4) == 0
    assert (c.N, c.H, c.D, c.cap, c.len, c.budget, c.offset, c.ring_head, c.step) == (2, 3, 64, 16, 8, 8, 4, 0, 0)
    assert init(C.byref(c), None, p, 2, 3, 64, 16, 8, 8, 4) == 1
    assert init(C.byref(c), p, p, 2, 3, 48, 16, 8, 8, 4) == 2
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 9, 8, 4) == 4      # len > budget
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 8, 17, 4) == 4     # budget > cap
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 0) == 4      # offset < 1
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 8) == 4      # offset > budget - 1
    assert init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 4) == 0
    ev = C.c_int(0)
    step = L.ec_decode_step
    assert step(None, p, p, C.byref(c), 1.0, p, C.byref(ev), None, p, 1 << 20, None) == 1
    assert step(p, p, p, C.byref(c), 0.0, p, C.byref(ev), None, p, 1 << 20, None) == 4
    assert step(p, p + 4, p, C.byref(c), 1.0, p, C.byref(ev), None, p, 1 << 20, None) == 3
    assert step(p, p, p, C.byref(c), 1.0, p, C.byref(ev), None, None, 0, None) == 5
    assert (c.len, c.ring_head, c.step) == (8, 0, 0)               # failed calls leave the state alone
    assert L.ec_decode_workspace(C.byref(c)) >= 256


def test_ratio_cache_init_validation(L):
    p = 0x10000
    c = ec.ec_cache()
    ring = (C.c_int * 8)()
    f = L.ec_cache_init_ratio
    assert f(C.byref(c), p, p, 1, 2, 64, 64, 20, 8, 0.5, 40, ring) == 0
    assert list(ring) == list(range(12, 20)) and c.policy == 1 and c.n_tot == 40 and c.len == 20
    assert f(C.byref(c), p, p, 1, 2, 64, 64, 20, 8, 0.5, 40, None) == 1       # ring missing
    assert f(C.byref(c), p, p, 1, 2, 64, 64, 6, 8, 0.5, 40, ring) == 4        # fewer rows than the offset
    assert f(C.byref(c), p, p, 1, 2, 64, 64, 20, 8, 0.0, 40, ring) == 4       # ratio out of range
    assert f(C.byref(c), p, p, 1, 2, 64, 64, 20, 8, 0.5, 10, ring) == 4       # fewer tokens seen than rows held


def test_statistic_prefix_and_from_lse_reject_bad_arguments_on_the_host(L):
    p = 0x10000
    ws = 1 << 20
    f = L.ec_importance_statistic
    assert f(p, None, p, None, 1, 1, 16, 0, 64, 1.0, 0, 0.0, p, ws, None) == 1            # NULL
    assert f(p, p, p, None, 1, 1, 0, 4, 64, 1.0, 0, 0.0, p, ws, None) == 2                # no query
    assert f(p, p, p, None, 1, 1, 16, -1, 64, 1.0, 0, 0.0, p, ws, None) == 2              # negative prefix
    assert f(p, p, p, None, 1, 1, 16, 16384, 64, 1.0, 0, 0.0, p, ws, None) == 2           # P + Tq too long
    assert f(p, p, p, None, 1, 1, 16, 0, 64, 1.0, 4, 0.0, p, ws, None) == 4               # unknown statistic
    assert f(p, p, p, None, 1, 1, 16, 0, 64, 1.0, 3, 0.0, p, ws, None) == 4               # beta outside (0, 1)
    assert f(p, p, p, None, 1, 1, 16, 0, 64, 1.0, 3, 1.0, p, ws, None) == 4
    assert f(p, p, p, p + 4, 1, 1, 16, 0, 64, 1.0, 1, 0.0, p, ws, None) == 3              # lse alignment
    assert f(p, p, p, None, 1, 1, 16, 0, 64, 1.0, 2, 0.0, p, 8, None) == 5                # workspace too small
    g = L.ec_importance_prefix
    assert g(p, p, None, None, 1, 1, 16, 3, 64, 1.0, p, ws, None) == 1
    assert g(p, p, p, None, 1, 1, 16, 3, 64, float("nan"), p, ws, None) == 4
    h = L.ec_importance_from_lse
    assert h(p, p, None, p, 1, 1, 16, 64, 1.0, p, ws, None) == 1                          # lse missing
    assert h(p, p, p, p, 1, 1, 16, 32, 1.0, p, ws, None) == 2


def test_prefill_attention_rejects_bad_arguments_on_the_host(L):
    p = 0x10000
    f = L.ec_prefill_attention
    ws = 1 << 20
    # (Q, K, V, out, lse, scores, N, H, Tq, P, D, scale, ws, ws_bytes, stream); nothing is launched on an error
    assert f(None, p, p, p, None, None, 1, 1, 16, 0, 64, 1.0, p, ws, None) == 1
    assert f(p, p, None, p, None, None, 1, 1, 16, 0, 64, 1.0, p, ws, None) == 1
    assert f(p, p, p, None, None, None, 1, 1, 16, 0, 64, 1.0, p, ws, None) == 1
    assert f(p, p, p, p, None, None, 1, 1, 16, 0, 48, 1.0, p, ws, None) == 2          # head dimension
    assert f(p, p, p, p, None, None, 1, 1, 0, 0, 64, 1.0, p, ws, None) == 2           # no queries
    assert f(p, p, p, p, None, None, 1, 1, 16, -1, 64, 1.0, p, ws, None) == 2         # negative prefix
    assert f(p, p, p, p, None, None, 1, 1, 16, 0, 64, 0.0, p, ws, None) == 4          # scale
    assert f(p, p, p + 8, p, None, None, 1, 1, 16, 0, 64, 1.0, p, ws, None) == 3      # V misaligned
    assert f(p, p, p, p, p + 4, None, 1, 1, 16, 0, 64, 1.0, p, ws, None) == 3         # lse misaligned
    assert f(p, p, p, p, None, None, 1, 1, 16, 0, 64, 1.0, None, 0, None) == 5
    assert f(p, p, p, p, None, None, 1, 1, 16, 0, 64, 1.0, p, 64, None) == 5          # workspace too small
    assert f(p, p, p, p, None, None, 1, 1, 16, 0, 64, 1.0, p + 16, ws, None) == 3     # workspace misaligned


def test_cache_concat_rejects_bad_arguments_on_the_host(L):
    p = 0x10000
    c = ec.ec_cache()
    assert L.ec_cache_init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 4) == 0
    f = L.ec_cache_concat
    assert f(C.byref(c), None, p, 4, p, p, None) == 1
    assert f(None, p, p, 4, p, p, None) == 1
    assert f(C.byref(c), p, p, 0, p, p, None) == 4                                        # no new rows
    assert f(C.byref(c), p, p + 2, 4, p, p, None) == 3
    c.ring_head = 4                                                                       # outside 0..offset-1
    assert f(C.byref(c), p, p, 4, p, p, None) == 4
    c.ring_head = 0
    c.len = 0                                                                             # nothing cached yet
    assert f(C.byref(c), p, p, 4, p, p, None) == 4
    ring = (C.c_int * 4)()
    r = ec.ec_cache()
    assert L.ec_cache_init_ratio(C.byref(r), p, p, 1, 2, 64, 64, 20, 4, 0.5, 40, ring) == 0
    assert f(C.byref(r), p, p, 4, p, p, None) == 4                                        # queue order not tracked


def test_select_compact_and_noalloc_validation(L):
    p = 0x10000
    ws = 1 << 20
    f = L.ec_select_compact
    assert f(p, p, p, 2, 4, 16, 64, 8, 3, 0, 0, p, p, 8, p, None, p, ws, None) == 4       # 8 units not a multiple of 3
    assert f(p, p, p, 2, 4, 16, 64, 8, 0, 0, 0, p, p, 8, p, None, p, ws, None) == 4       # share < 1
    assert f(p, p, p, 2, 4, 16, 64, 8, 4, 0, 2, p, p, 8, p, None, p, ws, None) == 4       # unknown compaction
    assert L.ec_select_compact_workspace(2, 4, 16, 64, 8, 4) >= 256 + 2 * 16 * 4
    assert L.ec_select_compact_workspace(2, 4, 16, 64, 8, 3) == 0
    assert L.ec_decode_noalloc_capacity() == 2 << 20
    big = ec.ec_cache()
    assert L.ec_cache_init(C.byref(big), p, p, 1024, 64, 128, 128, 128, 128, 16) == 0     # 65536 units
    assert L.ec_decode_workspace(C.byref(big)) > L.ec_decode_noalloc_capacity()
    ev = C.c_int(0)
    assert L.ec_decode_step_noalloc(p, p, p, C.byref(big), 1.0, p, C.byref(ev), None, None) == 8
    assert (big.len, big.step) == (128, 0)


def test_queue_order_tracking_validation(L):
    p = 0x10000
    c = ec.ec_cache()
    ring = (C.c_int * 8)()
    order = (C.c_int * 64)()
    assert L.ec_cache_init_ratio(C.byref(c), p, p, 1, 2, 64, 64, 20, 8, 0.5, 40, ring) == 0
    assert not c.queue_slots_host
    assert L.ec_cache_track_order(C.byref(c), None) == 1
    assert L.ec_cache_track_order(C.byref(c), order) == 0
    assert list(order)[:20] == list(range(20))
    c.step = 3
    assert L.ec_cache_track_order(C.byref(c), order) == 4            # rows may no longer be in slot order
    fixed = ec.ec_cache()
    assert L.ec_cache_init(C.byref(fixed), p, p, 1, 2, 64, 64, 20, 32, 8) == 0
    assert L.ec_cache_track_order(C.byref(fixed), order) == 4        # the fixed budget needs no list


def test_a_zeroed_or_damaged_cache_struct_is_an_error_not_a_crash(L):
    """The struct is caller-owned plain data: every call that reads one re-checks it."""
    p = 0x10000
    z = ec.ec_cache()                                   # all zero: N = H = 0 used to divide by zero
    assert L.ec_decode_workspace(C.byref(z)) == 0
    assert L.ec_decode_workspace(None) == 0
    ev = C.c_int(0)
    assert L.ec_decode_step_noalloc(p, p, p, C.byref(z), 1.0, p, C.byref(ev), None, None) == 1      # Kc, Vc NULL
    assert L.ec_decode_step(p, p, p, C.byref(z), 1.0, p, C.byref(ev), None, p, 1 << 20, None) == 1
    assert L.ec_decode_steps(p, p, p, 4, C.byref(z), 1.0, p, None, p, 1 << 20, None) == 1
    c = ec.ec_cache()
    assert L.ec_cache_init(C.byref(c), p, p, 2, 3, 64, 16, 8, 8, 4) == 0
    for field, bad, want in (("N", 0, 2), ("H", -1, 2), ("D", 96, 2), ("cap", 0, 2), ("budget", 17, 4),
                             ("ring_head", 4, 4), ("policy", 7, 4), ("offset", 0, 4), ("len", 9, 4)):
        good = getattr(c, field)
        setattr(c, field, bad)
        assert L.ec_decode_step(p, p, p, C.byref(c), 1.0, p, C.byref(ev), None, p, 1 << 20, None) == want, field
        assert L.ec_decode_step_noalloc(p, p, p, C.byref(c), 1.0, p, C.byref(ev), None, None) == want, field
        setattr(c, field, good)
    assert (c.len, c.step) == (8, 0)


def test_host_tensor_calls_validate_before_enqueueing_anything(L):
    """A rejected ec_compress_host / ec_decode_steps_host must not have started a copy: with no GPU in
    this process any enqueued copy would surface as EC_ERR_CUDA (6) instead of the argument's code."""
    p = 0x10000
    ws = 1 << 22
    f = L.ec_compress_host
    ok_args = [p, p, p, p, p, p, p, 1, 2, 16, 64, 1.0, 8, 0, 1, p, p, 8, p, None, p, ws, p, ws, None]

    def call(**change):
        a = list(ok_args)
        for k, v in change.items():
            a[int(k[1:])] = v
        return f(*a)

    assert call(a11=0.0) == 4                       # scale
    assert call(a12=17) == 4                        # n_keep > T
    assert call(a17=4) == 4                         # cap < n_keep
    assert call(a13=5) == 4                         # unknown population
    assert call(a21=0) == 5                         # importance workspace too small
    assert call(a23=0) == 5                         # selection workspace too small
    assert call(a20=p + 16) == 3                    # workspace not 256-byte aligned
    assert call(a3=p + 2) == 3                      # staging not 16-byte aligned
    c = ec.ec_cache()
    assert L.ec_cache_init(C.byref(c), p, p, 1, 2, 64, 16, 8, 8, 4) == 0
    g = L.ec_decode_steps_host
    one = 1
    assert g(p, p, p, p, p, p, p, p, 4, 2, C.byref(c), 0.0, p, ws, None, one, one) == 4      # scale
    assert g(p, p, p, p, p, p, p, p, 4, 2, C.byref(c), 1.0, p, 0, None, one, one) == 5       # workspace
    assert g(p, p, p, p, p, p + 8, p, p, 4, 2, C.byref(c), 1.0, p, ws, None, one, one) == 3  # staging alignment
    c.N = 0
    assert g(p, p, p, p, p, p, p, p, 4, 2, C.byref(c), 1.0, p, ws, None, one, one) == 2      # damaged struct
    c.N = 1
    assert (c.len, c.step) == (8, 0)


def test_header_is_plain_c(tmp_path):
    """ec.h is a C header: a C99 translation unit that includes nothing else compiles against it
    and can name every declared function with its declared type."""
    import subprocess
    names = _declared()
    src = tmp_path / "use_ec.c"
    body = "\n".join(f"    (void)&{n};" for n in names)
    src.write_text('#include "ec.h"\nint main(void)\n{\n    ec_cache c;\n    (void)sizeof(c);\n' + body +
                   "\n    return EC_OK;\n}\n")
    r = subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-fsyntax-only",
                        "-I", os.path.join(ROOT, "include"), str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
