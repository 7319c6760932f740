"""The C-ABI library loads, exports what include/stq.h declares, and its host-only logic works (no GPU)."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "stq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(stq_lib):
    names = declared_symbols()
    assert {"stq_create", "stq_destroy", "stq_init_state", "stq_step", "stq_layer_stats", "stq_repack",
            "stq_decide", "stq_step_host", "stq_grad_stats"} <= set(names)
    for n in names:
        assert hasattr(stq_lib, n), n


def test_struct_sizes_match_the_header(stq_lib):
    from paper_2604_06836_b200 import stq
    assert C.sizeof(stq.CTensor) == 120        # 10 pointers, numel, block, 4 widths, weight_decay, lp_dtype, param_lp, v_log, sr_id
    assert C.sizeof(stq.CHParams) == 88        # 4 doubles, step, 2 ints, 4 pointers, sr_seed
    assert C.sizeof(stq.CPolicyCfg) == 40


@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16, 32])
def test_buffer_sizes(stq_lib, O, bits):
    from paper_2604_06836_b200 import stq
    for n in (1, 7, 128, 129, 1000, 4096, 50257 * 1600):
        want = ((n * bits + 7) // 8 + 15) // 16 * 16
        assert stq.codes_bytes(n, bits) == want == O.codes_bytes(n, bits)
        for block in (128, 256, 512):
            assert stq.scales_bytes(n, block) == 4 * ((n + block - 1) // block) == 4 * O.num_blocks(n, block)


def test_errors_without_a_device_or_with_bad_arguments(stq_lib):
    from paper_2604_06836_b200 import stq
    assert stq_lib.stq_strerror(0) == b"ok"
    for code in range(-12, 0):
        assert stq_lib.stq_strerror(code) not in (b"ok", b"unknown error")
    h = C.c_void_p()
    assert stq_lib.stq_create(None, 0) == -1
    import torch
    if not torch.cuda.is_available():
        assert stq_lib.stq_create(C.byref(h), 0) == -7 and not h.value     # STQ_E_CUDA, nothing allocated
    assert stq_lib.stq_step(None, None, 0, None, 0, None) == -1
    cfg = stq.CPolicyCfg(0.1, 0.0, 1e-8, 10, 0, 0)
    p = C.c_void_p()
    assert stq_lib.stq_policy_create(C.byref(p), C.byref(cfg)) == -9       # tau must be positive


def test_policy_matches_oracle_on_random_statistics(stq_lib, O):
    from paper_2604_06836_b200 import stq
    rng = np.random.default_rng(0)
    for cv_signed in (False, True):
        pg = stq.Policy(alpha=0.1, tau=100.0, eps_stat=1e-8, interval=10, cv_of_signed=cv_signed)
        po = O.new_policy(0.1, 100.0, 1e-8, cv_of_signed=cv_signed)
        L = 150
        for t in [1, 2, 3, 4, 10, 20, 30, 500, 1000]:
            N = rng.integers(100, 10 ** 7, L).astype(np.float64)
            n = 10.0 ** rng.uniform(-6, -1, L)
            mu = n * rng.uniform(0.3, 0.99, L)
            stats = np.stack([rng.normal(0, 1, L) * mu * np.sqrt(N), mu * N, n * n * N, N], axis=1)
            stats[7] = [0.0, 0.0, 0.0, 1000.0]      # a dead layer
            assert pg.is_decision_step(t) == O.is_decision_step(t, 10)
            bg, sg = pg.decide(stats, t)
            bo, so = O.decide(po, stats, t)
            assert (bg == bo).all()
            fin = np.isfinite(so)
            np.testing.assert_allclose(sg[fin], so[fin], rtol=1e-12, atol=1e-12)
            assert (sg[~fin] == so[~fin]).all() and bg[7] == 4
            np.testing.assert_allclose(pg.state, [po.n_ema, po.r_ema, po.v_ema], rtol=1e-13)
    # checkpoint / resume of the three running averages
    saved = pg.state.copy()
    p2 = stq.Policy(alpha=0.1, tau=100.0, eps_stat=1e-8, interval=10, cv_of_signed=True)
    p2.state = saved
    b1, s1 = pg.decide(stats, 2000)
    b2, s2 = p2.decide(stats, 2000)
    assert (b1 == b2).all() and (s1 == s2).all()


def test_policy_schedule_and_anchor(stq_lib):
    from paper_2604_06836_b200 import stq
    p = stq.Policy(alpha=1.0, tau=1e-9, eps_stat=0.0, interval=7)
    assert [t for t in range(1, 30) if p.is_decision_step(t)] == [1, 2, 3, 4, 7, 14, 21, 28]
    N = 1000.0
    row = [0.0, 0.8e-3 * N, 1e-6 * N, N]
    bits, score = p.decide(np.array([row] * 5), 10 ** 6)
    assert np.allclose(score, 7.2, atol=1e-9) and (bits == 8).all()   # an average layer lands on 8 bits


def test_static_stats_binding_rejects_what_the_c_call_cannot_see():
    """The C entry point gets a pointer and a count; a gradient of another type or layout would be read as
    dense fp32 (twice the length of an fp16 buffer).  The binding refuses those before any launch."""
    import torch
    from paper_2604_06836_b200 import stq
    out = torch.zeros(4, dtype=torch.float64)
    for bad in (torch.zeros(64, dtype=torch.float16), torch.zeros(64, dtype=torch.float64),
                torch.zeros(64, dtype=torch.int32)):
        with pytest.raises(ValueError, match="float32 or bfloat16"):
            stq.grad_stats_static(bad, out)
    with pytest.raises(ValueError, match="contiguous"):
        stq.grad_stats_static(torch.zeros(8, 8)[:, ::2], out)
    with pytest.raises(ValueError, match="float64"):
        stq.grad_stats_static(torch.zeros(64), torch.zeros(4))
    with pytest.raises(ValueError, match="float64"):
        stq.grad_stats_static(torch.zeros(64), torch.zeros(3, dtype=torch.float64))
    with pytest.raises(ValueError, match="same CUDA device"):
        stq.grad_stats_static(torch.zeros(64), out)          # host tensors never reach the library
