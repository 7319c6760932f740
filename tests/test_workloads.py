"""The synthetic workloads: shape lists against the published sizes of the models they stand for,
and the seeded draws."""
import numpy as np
import pytest
import torch

from paper_2604_06836_b200 import workloads as W

# Published parameter counts of the architectures (tied output heads counted once).
PUBLISHED = {
    "cfg2": 124_439_808,           # GPT-2 small
    "gpt2_medium": 354_823_168,
    "cfg4": 774_030_080,           # GPT-2 large
    "cfg5": 1_557_611_200,         # GPT-2 XL
    "cfg3": 86_567_656,            # ViT-B/16, 1000 classes
    "vit_b32": 88_224_232,         # ViT-B/32, 1000 classes
    "roberta_large": 355_412_057,  # RoBERTa-Large with its masked-LM head
}


@pytest.mark.parametrize("name,count", sorted(PUBLISHED.items()))
def test_shape_lists_have_the_published_sizes(name, count):
    assert W.config(name).total_params == count


def test_draws_are_seeded_and_typed():
    w = W.scaled(W.config("gpt2_medium"), W.small_gpt2())
    a, b = W.draw_grad(w, 3, 7), W.draw_grad(w, 3, 7)
    assert a.dtype == torch.float16 and torch.equal(a, b)
    assert not torch.equal(a, W.draw_grad(w, 3, 8))
    # the loss scale multiplies the draw before the rounding to fp16
    plain = W.draw_grad(W.scaled(W.config("cfg2"), W.small_gpt2()), 3, 7)
    assert plain.dtype == torch.float32
    w32 = W.scaled(W.config("gpt2_medium"), W.small_gpt2())
    assert w32.loss_scale == 4096.0 and w32.lp_copy == "fp16"
    x = a.float() / w.loss_scale
    assert torch.isfinite(x).all() and float(x.abs().max()) > 0


def test_mixed_widths_land_on_the_requested_mean():
    for name in ("cfg2", "cfg5", "roberta_large"):
        w = W.config(name)
        bm, bv, _ = W.draw_bits(w)
        assert w.bits_mean[0] <= W.mean_bits(w, bm, bv) <= w.bits_mean[1]
        assert set(np.unique(bm)) <= set(W.WIDTH_SET) and set(np.unique(bv)) <= set(W.WIDTH_SET)


# bytes per step by the roofline's definition, worked out per parameter: parameter read and written (8), gradient
# (4 fp32, 2 bf16), codes of both states read and written, 16 bytes of block scales per block
ALGORITHMIC = {
    "cfg2": (4, 128, 1_824_604_320),
    "cfg3": (4, 256, 1_267_223_944),
    "cfg4": (2, 128, 9_919_307_680),
    "cfg5": (2, 128, 19_636_028_912),      # 12.6065 bytes per parameter
}


@pytest.mark.parametrize("name", sorted(ALGORITHMIC))
def test_algorithmic_bytes_follow_the_per_parameter_formula(name):
    from paper_2604_06836_b200.runner import algorithmic_bytes
    gb, block, want = ALGORITHMIC[name]
    w = W.config(name)
    bm, bv, _ = W.draw_bits(w)
    got = algorithmic_bytes(w.numels, bm, bv, w.block, w.grad_dtype, bool(w.lp_copy))
    assert got == want
    n = np.array(w.numels, dtype=np.float64)
    formula = float((n * (8 + gb + 2 * (bm.astype(np.float64) + bv) / 8 + 16.0 / block)).sum())
    assert abs(got - formula) <= 16 * len(w.numels)        # only whole bytes and short last blocks differ
    if name == "cfg5":
        assert abs(got / w.total_params - 12.6065) < 1e-4


def test_algorithmic_bytes_count_both_scale_vectors_and_none_at_32_bits():
    from paper_2604_06836_b200.runner import algorithmic_bytes
    n = 1 << 20
    base = n * (8 + 4)
    assert algorithmic_bytes([n], [4], [4], 128, "fp32") == base + 2 * (n // 2 + n // 2) + 16 * (n // 128)
    assert algorithmic_bytes([n], [32], [4], 128, "fp32") == base + 2 * (4 * n + n // 2) + 8 * (n // 128)
    assert algorithmic_bytes([n], [32], [32], 128, "fp32") == base + 2 * (8 * n)
    assert algorithmic_bytes([n], np.array([8], np.uint8), np.array([8], np.uint8), 256, "bf16", True) == \
        n * (8 + 2 + 2) + 2 * (2 * n) + 16 * (n // 256)
    assert algorithmic_bytes([130], [3], [2], 128, "bf16") == 130 * 10 + 2 * (49 + 33) + 16 * 2
    assert algorithmic_bytes([n], [4], [4], 128, "fp32", False, 2) == base + 2 * (n // 2 + n // 2) + 24 * (n // 128)
