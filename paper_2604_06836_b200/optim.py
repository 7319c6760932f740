"""Algorithm 1 as a ``torch.optim.Optimizer``: AdamW whose moments live in the packed, per-tensor
mixed-width state of libstq, with the paper's transition decision choosing the widths.

This module only arranges buffers and calls: the update, the quantizers and the statistics run in
the CUDA library, the decision in its host policy.  One optimizer step is

    decision step (t mod U == 0 or t < 5):
        stq_grad_stats -> stq_layer_stats -> stq_decide      (statistics of the fresh gradients)
        stq_step with bits_*_out = the new widths            (the same step writes the new widths)
    other steps:
        stq_step in place

which is the order Algorithm 1 prints.  With ``order="fused"`` the statistics ride on the update of
the step before a decision step instead (``STQ_WITH_STATS``), which saves the extra pass over the
gradients.  Every tensor starts at ``init_bits`` (16 in the paper).
"""
from __future__ import annotations

from typing import Iterable

import numpy as np
import torch

from . import stq


class STQAdamW(torch.optim.Optimizer):
    """AdamW with block-quantized moments at per-tensor, per-step bit-widths (STQuant, Algorithm 1).

    params: fp32 CUDA tensors (or param groups; ``lr`` and ``weight_decay`` may differ per group,
    the other hyper-parameters are shared).  Gradients may be fp32, bf16 or fp16, one type for all.
    policy: "paper" lets the transition decision pick widths in {4, 8, 16, 32} every ``interval`` steps
    (and while t < 5); "fixed" keeps ``init_bits`` (an int, or a pair (bits_m, bits_v)) for good.
    order: "paper" takes the statistics of a decision step from that step's own gradients in a pass
    before the update (Algorithm 1 as printed, one more read of the gradients on decision steps);
    "fused" lets them ride on the update of the step before (no extra pass; the decision then sees
    gradients that are one step old, except at t = 1).
    v_log: the code of the second moment: "poly" (default) or "pl" (they differ at 8 and 16 bits), "sr"
    (stochastic rounding; ``self.sr_seed`` seeds its random words) or "ts" (two scales per block).
    grad_scaler_inv / found_inf: optional one-element float32 CUDA tensors for loss-scaled training.
    With ``found_inf`` set, ``step()`` reads it on the host first (one small synchronising copy): a step
    with a non-finite gradient is left out entirely, so the step count t, the bias corrections and the
    decision schedule follow the steps actually taken and no statistics of a skipped step reach the policy.
    """

    def __init__(self, params: Iterable, lr: float = 1e-3, betas=(0.9, 0.999), eps: float = 1e-8,
                 weight_decay: float = 0.01, *, block: int = 128, init_bits=16, policy: str = "paper",
                 interval: int = 10, alpha: float = 0.1, tau: float = 100.0, eps_stat: float = 1e-8,
                 v_log: str = "poly", decoupled_weight_decay: bool = True, order: str = "paper"):
        if policy not in ("paper", "fixed"):
            raise ValueError("policy is 'paper' or 'fixed'")
        if order not in ("paper", "fused"):
            raise ValueError("order is 'paper' or 'fused'")
        self.order = order
        self._carried_stats = None        # sums that rode on the last step (fused order), fetched right after it
        if block not in (32, 64, 128, 256, 512, 1024):
            raise ValueError("block is a power of two in 32..1024")
        defaults = dict(lr=lr, weight_decay=weight_decay)
        super().__init__(params, defaults)
        self.betas, self.eps = (float(betas[0]), float(betas[1])), float(eps)
        self.block, self.policy_kind, self.interval = block, policy, int(interval)
        self.decoupled = bool(decoupled_weight_decay)
        if v_log not in stq.VLOG_BY_NAME:
            raise ValueError("v_log is one of " + ", ".join(stq.VLOG_BY_NAME))
        self.v_log = stq.VLOG_BY_NAME[v_log]
        self.sr_seed = 0
        bm, bv = (init_bits, init_bits) if isinstance(init_bits, int) else init_bits
        self._params = [p for g in self.param_groups for p in g["params"]]
        if not self._params:
            raise ValueError("no parameters")
        dev = self._params[0].device
        for p in self._params:
            if p.device != dev or p.device.type != "cuda" or p.dtype != torch.float32 or not p.is_contiguous():
                raise ValueError("STQAdamW needs contiguous fp32 parameters on one CUDA device")
        self.device = dev
        self.handle = stq.Handle(dev.index if dev.index is not None else torch.cuda.current_device())
        self.policy = stq.Policy(alpha=alpha, tau=tau, eps_stat=eps_stat, interval=self.interval)
        self.bits_m = np.full(len(self._params), bm, dtype=np.uint8)
        self.bits_v = np.full(len(self._params), bv, dtype=np.uint8)
        self.states = [stq.alloc_state(p.numel(), block, int(bm), int(bv), dev, self.v_log) for p in self._params]
        self.t = 0
        self.skipped_steps = 0
        self.last_scores = None
        self.grad_scaler_inv = None      # torch tensor [1] float32 on the device, or None
        self.found_inf = None
        self.handle.init_state(stq.table([stq.make_row(p.numel(), block, None, s)
                                          for p, s in zip(self._params, self.states)]))
        self._tbl = None
        self._tbl_key = None

    # ---- tables ------------------------------------------------------------------------------------
    def _rows(self, states_out):
        rows = []
        k = 0
        for g in self.param_groups:
            lr_ratio = g["lr"] / self.param_groups[0]["lr"] if self.param_groups[0]["lr"] else 1.0
            if abs(lr_ratio - 1.0) > 0:
                raise ValueError("one learning rate per step() call: give every group the same lr, or use one "
                                 "optimizer per group")
            for p in g["params"]:
                grad = p.grad
                if grad is None:
                    raise ValueError("every parameter needs a gradient (frozen parameters do not belong here)")
                if not grad.is_contiguous():
                    grad = grad.contiguous()
                    p.grad = grad
                rows.append(stq.make_row(p.numel(), self.block, self.states[k], states_out[k], p.data, grad,
                                         g["weight_decay"], sr_id=k))
                k += 1
        return rows

    def _grad_dtype(self) -> int:
        kinds = {p.grad.dtype for p in self._params}
        if len(kinds) != 1:
            raise ValueError("all gradients must have one dtype")
        return stq.grad_dtype_of(self._params[0].grad)

    def _table(self):
        key = tuple((p.data_ptr(), p.grad.data_ptr()) for p in self._params) + tuple(
            g["weight_decay"] for g in self.param_groups)
        if self._tbl is None or key != self._tbl_key:
            self._tbl = stq.table(self._rows(self.states))
            self._tbl_key = key
        return self._tbl

    # ---- the step -----------------------------------------------------------------------------------
    @torch.no_grad()
    def step(self, closure=None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        if self.found_inf is not None and float(self.found_inf.item()) != 0.0:
            self.skipped_steps += 1       # nothing is launched, t does not advance, carried statistics are kept
            return loss
        self.t += 1
        t = self.t
        hp = dict(lr=self.param_groups[0]["lr"], beta1=self.betas[0], beta2=self.betas[1], eps=self.eps, t=t,
                  grad_dtype=self._grad_dtype(), decoupled_wd=self.decoupled,
                  inv_grad_scale=self.grad_scaler_inv, found_inf=self.found_inf, sr_seed=self.sr_seed)
        new_m = new_v = None
        if self.policy_kind == "paper" and self.policy.is_decision_step(t):
            stats, self._carried_stats = self._carried_stats, None    # fused order: they rode on the previous step
            if stats is None:
                tbl = self._table()
                self.handle.grad_stats(tbl, hp["grad_dtype"])
                stats = self.handle.layer_stats(len(self._params))
                if self.grad_scaler_inv is not None:   # the pre-pass sees the scaled gradients: unscale the sums
                    s = float(self.grad_scaler_inv.item())
                    stats[:, 0:2] *= s
                    stats[:, 2] *= s * s
            bits, self.last_scores = self.policy.decide(stats, t)
            new_m = new_v = bits                       # Algorithm 1: one width per layer for both states
        # fused order: if the next step decides, this one carries the statistics
        flags = stq.WITH_STATS if (self.order == "fused" and self.policy_kind == "paper" and
                                   self.policy.is_decision_step(t + 1)) else 0
        if new_m is None or ((new_m == self.bits_m).all() and (new_v == self.bits_v).all()):
            self.handle.step(self._table(), flags=flags, **hp)
            self._fetch_carried(flags)
            return loss
        out = []
        for k, p in enumerate(self._params):
            old = self.states[k]
            bm, bv = int(new_m[k]), int(new_v[k])
            if bm == old.bits_m and bv == old.bits_v:
                out.append(old)
                continue
            n = p.numel()
            mc, ms = (old.m_codes, old.m_scales) if bm == old.bits_m else (
                stq.alloc_codes(n, bm, self.device), stq.alloc_scales(n, bm, self.block, self.device))
            vc, vs = (old.v_codes, old.v_scales) if bv == old.bits_v else (
                stq.alloc_codes(n, bv, self.device), stq.alloc_scales(n, bv, self.block, self.device, self.v_log))
            out.append(stq.QState(mc, ms, bm, vc, vs, bv, self.v_log))
        self.handle.step(stq.table(self._rows(out)), flags=flags, **hp)
        self._fetch_carried(flags)
        torch.cuda.current_stream(self.device).synchronize()     # the old buffers are released below
        self.states = out
        self.bits_m, self.bits_v = np.array(new_m, np.uint8), np.array(new_v, np.uint8)
        self._tbl = None
        return loss

    def _fetch_carried(self, flags: int):
        # The sums are finished with the table they were taken with, and the next step's table may differ
        # (fresh gradient buffers), so they are brought to the host right away.
        if flags:
            self._carried_stats = self.handle.layer_stats(len(self._params))

    # ---- bookkeeping --------------------------------------------------------------------------------
    def state_bytes(self) -> int:
        return int(sum(s.m_codes.numel() + s.v_codes.numel() + 4 * (s.m_scales.numel() + s.v_scales.numel())
                       for s in self.states))

    def mean_bits(self) -> float:
        n = np.array([p.numel() for p in self._params], dtype=np.float64)
        return float((n * (self.bits_m.astype(np.float64) + self.bits_v) / 2).sum() / n.sum())

    def state_dict(self):
        d = super().state_dict()
        d["stq"] = dict(t=self.t, bits_m=self.bits_m.copy(), bits_v=self.bits_v.copy(), v_log=self.v_log,
                        block=self.block, policy=self.policy.state.copy(), sr_seed=self.sr_seed,
                        carried_stats=None if self._carried_stats is None else self._carried_stats.copy(),
                        states=[dict(m_codes=s.m_codes.clone(), m_scales=s.m_scales.clone(),
                                     v_codes=s.v_codes.clone(), v_scales=s.v_scales.clone()) for s in self.states])
        return d

    def load_state_dict(self, d):
        d = dict(d)
        q = d.pop("stq")
        super().load_state_dict(d)
        if q["block"] != self.block or q["v_log"] != self.v_log or len(q["states"]) != len(self._params):
            raise ValueError("state was written with another block size, v code variant or parameter list")
        self.t = int(q["t"])
        self.bits_m, self.bits_v = np.array(q["bits_m"], np.uint8), np.array(q["bits_v"], np.uint8)
        self.policy.state = q["policy"]
        self.sr_seed = int(q.get("sr_seed", self.sr_seed))
        carried = q.get("carried_stats")
        self._carried_stats = None if carried is None else np.array(carried, dtype=np.float64)
        self.states = [stq.QState(s["m_codes"].to(self.device).clone(), s["m_scales"].to(self.device).clone(), int(bm),
                                  s["v_codes"].to(self.device).clone(), s["v_scales"].to(self.device).clone(), int(bv),
                                  self.v_log)
                       for s, bm, bv in zip(q["states"], self.bits_m, self.bits_v)]
        self._tbl = None
