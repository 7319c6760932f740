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
