"""Synthetic, seeded stand-ins for the paper's GPT-2 / ViT optimizer workloads.

This module only describes shapes and draws random inputs (parameters, gradients, per-tensor
bit-widths).  It holds none of the optimizer's or quantizer's arithmetic, so the CUDA path and
the test oracle can both be fed from it without sharing any of the method's code.

The paper trains GPT-2 and ViT models on public corpora (Sec. 4, Table 1); the optimizer step only
sees tensors of the right shapes and value distributions, so seeded synthetic tensors stand in
for those runs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace

import numpy as np
import torch

WIDTH_SET = (2, 3, 4, 8, 16)
WIDTH_PROBS = (0.10, 0.20, 0.42, 0.22, 0.06)   # numel-weighted mean lands near 5.1 bits


# --------------------------------------------------------------------------------------------
# parameter-tensor shapes
# --------------------------------------------------------------------------------------------
def transformer_block_shapes(prefix: str, d: int, d_ff: int) -> list[tuple[str, tuple[int, ...]]]:
    return [
        (f"{prefix}.ln1.w", (d,)), (f"{prefix}.ln1.b", (d,)),
        (f"{prefix}.qkv.w", (d, 3 * d)), (f"{prefix}.qkv.b", (3 * d,)),
        (f"{prefix}.proj.w", (d, d)), (f"{prefix}.proj.b", (d,)),
        (f"{prefix}.ln2.w", (d,)), (f"{prefix}.ln2.b", (d,)),
        (f"{prefix}.fc.w", (d, d_ff)), (f"{prefix}.fc.b", (d_ff,)),
        (f"{prefix}.fcproj.w", (d_ff, d)), (f"{prefix}.fcproj.b", (d,)),
    ]


def gpt2_shapes(n_layer: int, d: int, vocab: int = 50257, ctx: int = 1024):
    """GPT-2 family: tied output head, so wte appears once."""
    s = [("wte", (vocab, d)), ("wpe", (ctx, d))]
    for l in range(n_layer):
        s += transformer_block_shapes(f"h{l}", d, 4 * d)
    s += [("lnf.w", (d,)), ("lnf.b", (d,))]
    return s


def vit_shapes(n_layer: int = 12, d: int = 768, d_ff: int = 3072, patch: int = 16, chans: int = 3,
               tokens: int = 197, classes: int = 1000):
    s = [("patch.w", (d, chans, patch, patch)), ("patch.b", (d,)), ("cls", (d,)), ("pos", (tokens, d))]
    for l in range(n_layer):
        s += transformer_block_shapes(f"b{l}", d, d_ff)
    s += [("norm.w", (d,)), ("norm.b", (d,)), ("head.w", (classes, d)), ("head.b", (classes,))]
    return s


def roberta_shapes(n_layer: int = 24, d: int = 1024, vocab: int = 50265, positions: int = 514):
    """RoBERTa (Table 1 fine-tunes RoBERTa-Large): embeddings with their norm, encoder blocks, and the
    masked-LM head (dense, norm, output bias; the decoder matrix is tied to the word embeddings)."""
    s = [("emb.word", (vocab, d)), ("emb.pos", (positions, d)), ("emb.type", (1, d)),
         ("emb.ln.w", (d,)), ("emb.ln.b", (d,))]
    for l in range(n_layer):
        s += transformer_block_shapes(f"l{l}", d, 4 * d)
    s += [("head.dense.w", (d, d)), ("head.dense.b", (d,)), ("head.ln.w", (d,)), ("head.ln.b", (d,)),
          ("head.bias", (vocab,))]
    return s


# --------------------------------------------------------------------------------------------
# workload configurations
# --------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    shapes: tuple                      # ((name, shape), ...)
    block: int
    grad_dtype: str                    # "fp32" | "bf16" | "fp16"
    grad_kind: str                     # "normal" | "student_t" | "normal_outliers"
    nu: int = 0                        # Student-t degrees of freedom
    scale_log10: tuple = (-3.0, -3.0)  # per-tensor scale is 10^U(lo, hi)
    bits_kind: str = "mixed"           # "fixed" | "mixed" | "m48_v348"
    bits_fixed: tuple = (8, 4)
    bits_mean: tuple = (5.0, 5.2)      # accepted numel-weighted mean for "mixed"
    steps: int = 1
    decision_interval: int = 10        # K (the paper's U)
    churn: float = 0.0                 # fraction of tensors whose width changes per decision step
    warmup_fp32_steps: int = 0
    seed: int = 0
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    loss_scale: float = 0.0            # > 0: gradients arrive multiplied by it (fp16 training)
    lp_copy: str = ""                  # "bf16" | "fp16": the step also writes the model's working copy
    v_log: str = "poly"                # code of the second moment: "poly" | "pl" (differ at widths 8 and 16) | "sr"
                                       # (stochastic rounding) | "ts" (two scales per block)

    @property
    def numels(self) -> list[int]:
        return [int(np.prod(s)) for _, s in self.shapes]

    @property
    def total_params(self) -> int:
        return int(sum(self.numels))


def config(name: str) -> Workload:
    """The five benchmark configurations, at full size."""
    if name == "cfg1":
        return Workload("cfg1-single-1M-m8v4", (("w", (1 << 20,)),), 128, "fp32", "normal",
                        scale_log10=(-3.0, -3.0), bits_kind="fixed", bits_fixed=(8, 4), steps=1,
                        decision_interval=1, warmup_fp32_steps=10, seed=0)
    if name == "cfg2":
        return Workload("cfg2-gpt2-small-124M", tuple(gpt2_shapes(12, 768)), 128, "fp32", "student_t",
                        nu=4, scale_log10=(-5.0, -2.0), steps=100, decision_interval=10, seed=2)
    if name == "cfg3":
        return Workload("cfg3-vit-b16-86M", tuple(vit_shapes()), 256, "fp32", "normal_outliers",
                        scale_log10=(-6.0, -3.0), steps=100, decision_interval=20, churn=0.10, seed=3)
    if name == "cfg4":
        return Workload("cfg4-gpt2-large-774M", tuple(gpt2_shapes(36, 1280)), 128, "bf16", "student_t",
                        nu=3, scale_log10=(-5.0, -2.0), bits_kind="m48_v348", steps=50,
                        decision_interval=10, seed=4)
    if name == "cfg5":
        return Workload("cfg5-gpt2-xl-1.5B", tuple(gpt2_shapes(48, 1600)), 128, "bf16", "student_t",
                        nu=3, scale_log10=(-5.0, -2.0), bits_mean=(4.9, 5.1), steps=20,
                        decision_interval=5, seed=5)
    if name == "cfg5s":   # the cfg5 recipe on 6 of the 48 layers: small enough for a full profiler capture
        return Workload("cfg5s-gpt2-xl-6-layers", tuple(gpt2_shapes(6, 1600)), 128, "bf16", "student_t",
                        nu=3, scale_log10=(-5.0, -2.0), bits_mean=(4.9, 5.1), steps=20,
                        decision_interval=5, seed=5)
    # Table 1's other models, trained the way Sec. 4 describes (fp16 with a loss scale): fp16 gradients
    # times 2^12, unscaled inside the step, and an fp16 working copy of the parameters written by it.
    amp = dict(block=128, grad_dtype="fp16", grad_kind="student_t", nu=4, scale_log10=(-5.0, -2.0),
               steps=20, decision_interval=10, loss_scale=4096.0, lp_copy="fp16")
    if name == "gpt2_medium":
        return Workload("gpt2-medium-355M-fp16", tuple(gpt2_shapes(24, 1024)), seed=6, **amp)
    if name == "roberta_large":
        return Workload("roberta-large-356M-fp16", tuple(roberta_shapes()), seed=7, **amp)
    if name == "vit_b32":
        return Workload("vit-b32-88M-fp16", tuple(vit_shapes(patch=32, tokens=50)), seed=8, **amp)
    if name.startswith("pair-"):
        # one width pair on one large tensor ("pair-4-8": m at 4 bits, v at 8 bits; "pair-4-8-25": 2^25 elements):
        # isolates one fused body of the step kernel for per-body throughput and profiler counters
        parts = name.split("-")
        bm, bv = int(parts[1]), int(parts[2])
        lg = int(parts[3]) if len(parts) > 3 else 27
        return Workload(name, (("w", (1 << lg,)),), 128, "bf16", "student_t", nu=3, scale_log10=(-3.0, -3.0),
                        bits_kind="fixed", bits_fixed=(bm, bv), steps=20, decision_interval=1 << 30, seed=1)
    raise KeyError(name)


def scaled(w: Workload, shapes, steps: int | None = None) -> Workload:
    """Same recipe on a smaller shape list (for tests the oracle must finish in seconds)."""
    return replace(w, name=w.name + "-scaled", shapes=tuple(shapes), steps=w.steps if steps is None else steps)


# --------------------------------------------------------------------------------------------
# seeded draws
# --------------------------------------------------------------------------------------------
def draw_bits(w: Workload) -> tuple[np.ndarray, np.ndarray, int]:
    """Per-tensor stored widths (bits_m[L], bits_v[L]) and the reseed count used."""
    L = len(w.shapes)
    numel = np.asarray(w.numels, dtype=np.float64)
    if w.bits_kind == "fixed":
        return (np.full(L, w.bits_fixed[0], np.uint8), np.full(L, w.bits_fixed[1], np.uint8), 0)
    if w.bits_kind == "m48_v348":
        rng = np.random.RandomState(w.seed)
        return (rng.choice([4, 8], size=L).astype(np.uint8), rng.choice([3, 4, 8], size=L).astype(np.uint8), 0)
    for k in range(10000):
        rng = np.random.RandomState(w.seed + k)
        bm = rng.choice(WIDTH_SET, size=L, p=WIDTH_PROBS).astype(np.uint8)
        bv = rng.choice(WIDTH_SET, size=L, p=WIDTH_PROBS).astype(np.uint8)
        mean = float((numel * (bm.astype(np.float64) + bv) / 2).sum() / numel.sum())
        if w.bits_mean[0] <= mean <= w.bits_mean[1]:
            return bm, bv, k
    raise RuntimeError("no seed gives the requested mean width")


def mean_bits(w: Workload, bm: np.ndarray, bv: np.ndarray) -> float:
    numel = np.asarray(w.numels, dtype=np.float64)
    return float((numel * (bm.astype(np.float64) + bv) / 2).sum() / numel.sum())


def churn_bits(w: Workload, bm: np.ndarray, bv: np.ndarray, decision_index: int):
    """Seeded width change for ``churn`` of the tensors (both states get a width != the old one)."""
    L = len(bm)
    rng = np.random.RandomState(w.seed * 7919 + 104729 * (decision_index + 1))
    k = max(1, int(round(w.churn * L))) if w.churn > 0 else 0
    idx = rng.choice(L, size=k, replace=False)
    bm, bv = bm.copy(), bv.copy()
    for i in idx:
        bm[i] = rng.choice([b for b in WIDTH_SET if b != bm[i]])
        bv[i] = rng.choice([b for b in WIDTH_SET if b != bv[i]])
    return bm, bv, np.sort(idx)


def tensor_scales(w: Workload) -> np.ndarray:
    rng = np.random.RandomState(w.seed + 99991)
    lo, hi = w.scale_log10
    return 10.0 ** rng.uniform(lo, hi, size=len(w.shapes))


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def draw_param(w: Workload, idx: int, device="cpu") -> torch.Tensor:
    """fp32 master parameters ~ N(0, 0.02), flattened."""
    n = w.numels[idx]
    g = _gen(device, 1000 + 7 * w.seed + 1000003 * idx)
    return torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 0.02, generator=g)


def draw_grad(w: Workload, idx: int, step: int, device="cpu", scale: float | None = None,
              chunk: int = 1 << 24) -> torch.Tensor:
    """Gradient of tensor ``idx`` at ``step`` (flattened; fp32, bf16 or fp16 per the workload; times the
    workload's loss scale when it has one)."""
    n = w.numels[idx]
    if scale is None:
        scale = float(tensor_scales(w)[idx])
    g = _gen(device, 17 + 31 * w.seed + 1000003 * idx + 7919 * step)
    out = torch.empty(n, dtype=torch.float32, device=device)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        z = torch.empty(m, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g)
        if w.grad_kind == "student_t":
            s = torch.zeros(m, dtype=torch.float32, device=device)
            for _ in range(w.nu):
                s += torch.empty(m, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g) ** 2
            z = z / torch.sqrt(s / w.nu)
        elif w.grad_kind == "normal_outliers":
            mask = torch.empty(m, dtype=torch.float32, device=device).uniform_(0.0, 1.0, generator=g) < 1e-3
            z = torch.where(mask, torch.sign(z) * 100.0, z)
        out[lo:lo + m] = z * scale
    if w.loss_scale > 0:
        out *= w.loss_scale
    if w.grad_dtype == "bf16":
        return out.to(torch.bfloat16)
    return out.to(torch.float16) if w.grad_dtype == "fp16" else out


def small_gpt2(d: int = 200, n_layer: int = 2, vocab: int = 1031, ctx: int = 64):
    """A GPT-2-shaped list small enough for element-by-element oracle checks, with ragged tails."""
    return gpt2_shapes(n_layer, d, vocab, ctx)


def small_vit(d: int = 136, n_layer: int = 2, d_ff: int = 520, classes: int = 250):
    return vit_shapes(n_layer, d, d_ff, patch=4, chans=3, tokens=17, classes=classes)
