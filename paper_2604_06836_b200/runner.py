"""Device-side driver of a workload: allocates the tensors, builds the stq table, steps.

Everything numerical happens inside libstq; this module only owns buffers (through torch) and
keeps the per-tensor widths.  Used by the benchmark, the smoke check and the GPU tests.
"""
from __future__ import annotations

from typing import Sequence

import numpy as np
import torch

from . import stq
from .workloads import Workload, draw_grad, draw_param, tensor_scales


def _round_up(x: int, a: int) -> int:
    return (x + a - 1) // a * a


def algorithmic_bytes(numels, bits_m, bits_v, block: int, grad_dtype: str, lp_copy: bool = False,
                      v_scales_per_block: int = 1) -> int:
    """Bytes one step must move over a parameter list: per element the parameter read and written (8),
    the gradient (4 for fp32, 2 for bf16 / fp16), the codes of both states read and written
    (2 * (b_m + b_v) / 8), the working copy if any (2); per block the fp32 scales of both states read and
    written (16; a 32-bit state has none; the two-scale code of v keeps two per block).  Code bytes are whole bytes per tensor, blocks include a short
    last one.  This is the numerator of the HBM roofline the benchmark reports."""
    gb = 4 if grad_dtype == "fp32" else 2
    gb += 2 if lp_copy else 0
    total = 0
    for n, bm, bv in zip(numels, bits_m, bits_v):
        n, bm, bv = int(n), int(bm), int(bv)
        nb = (n + block - 1) // block
        total += n * (8 + gb) + 2 * ((n * bm + 7) // 8 + (n * bv + 7) // 8)
        total += 4 * nb * (int(bm != 32) + v_scales_per_block * int(bv != 32)) * 2
    return int(total)


class Job:
    """Parameters, gradients and quantized AdamW state of one workload on one device."""

    def __init__(self, w: Workload, bits_m: Sequence[int], bits_v: Sequence[int], device="cuda",
                 handle: stq.Handle | None = None, draw_params: bool = True, tile_padded: bool = False):
        """tile_padded: every tensor's storage (parameters, gradients, codes, scales) is padded with zeros to a
        whole number of 4096-element tiles and the library is given the padded length, so that a step has no
        ragged last tiles (and hence a single launch).  The padding stays zero under the update (zero gradient,
        zero moments, zero parameter), adds nothing to the gradient sums and leaves the block maxima of the
        real elements as they are; ``params`` / ``grads`` remain views of the real elements."""
        self.w = w
        self.device = torch.device(device)
        self.handle = handle or stq.Handle(self.device.index if self.device.index is not None else torch.cuda.current_device())
        self.numels = w.numels
        self.tile_padded = bool(tile_padded)
        if tile_padded and w.v_log == "ts" and any(n % w.block for n in w.numels):
            # the two-scale code also keeps the block minimum, which zero padding inside a block would change
            raise ValueError("tile-padded storage with the two-scale code needs tensors of whole blocks")
        # the length the library is told: the real one, or the padded one
        self.tab_numels = [_round_up(n, stq.TILE) if tile_padded else n for n in self.numels]
        self.L = len(self.numels)
        self.block = w.block
        self.gdt = {"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}[w.grad_dtype]
        self.grad_dtype = {"fp32": stq.GRAD_F32, "bf16": stq.GRAD_BF16, "fp16": stq.GRAD_F16}[w.grad_dtype]
        self.scales = tensor_scales(w)
        # parameters and gradients live in two flat buffers; every tensor starts 256-byte aligned
        offs, total = [], 0
        for n in self.tab_numels:
            offs.append(total)
            total += _round_up(n, 64)
        self.offsets = offs
        self.param_flat = torch.zeros(total, dtype=torch.float32, device=self.device)
        self.grad_flat = torch.zeros(total, dtype=self.gdt, device=self.device)
        self.params = [self.param_flat[o:o + n] for o, n in zip(offs, self.numels)]
        self.grads = [self.grad_flat[o:o + n] for o, n in zip(offs, self.numels)]
        # loss-scaled training: 1/scale and the found-inf flag are read by the kernel from device memory
        self.inv_scale = (torch.tensor([1.0 / w.loss_scale], dtype=torch.float32, device=self.device)
                          if w.loss_scale > 0 else None)
        self.found_inf = torch.zeros(1, dtype=torch.float32, device=self.device) if w.loss_scale > 0 else None
        self.lp_flat = (torch.zeros(total, dtype={"bf16": torch.bfloat16, "fp16": torch.float16}[w.lp_copy],
                                    device=self.device) if w.lp_copy else None)
        self.params_lp = ([self.lp_flat[o:o + n] for o, n in zip(offs, self.numels)]
                          if w.lp_copy else [None] * self.L)
        if draw_params:
            for i in range(self.L):
                self.params[i].copy_(draw_param(w, i, self.device))
        self.bits_m = np.asarray(bits_m, dtype=np.uint8).copy()
        self.bits_v = np.asarray(bits_v, dtype=np.uint8).copy()
        self.v_log = stq.VLOG_BY_NAME[w.v_log]
        self.sr_seed = 0x5EED0000 + w.seed          # random words of the stochastic-rounding code
        self.states = [stq.alloc_state(n, self.block, int(bm), int(bv), self.device, self.v_log)
                       for n, bm, bv in zip(self.tab_numels, self.bits_m, self.bits_v)]
        self.wd = [w.weight_decay] * self.L
        self._tbl = None
        self.t = 0
        self.handle.init_state(self._make_table(self.states, self.states, with_inputs=False))
        self._tbl = None

    # ---- tables ----------------------------------------------------------------------------------
    def _make_table(self, st_in, st_out, with_inputs=True):
        rows = [stq.make_row(n, self.block, si if with_inputs else None, so,
                             self.params[i] if with_inputs else None,
                             self.grads[i] if with_inputs else None, self.wd[i],
                             self.params_lp[i] if with_inputs else None, sr_id=i)
                for i, (n, si, so) in enumerate(zip(self.tab_numels, st_in, st_out))]
        return stq.table(rows)

    def table(self):
        """In-place table at the current widths (cached until the widths change)."""
        if self._tbl is None:
            self._tbl = self._make_table(self.states, self.states)
        return self._tbl

    # ---- inputs ----------------------------------------------------------------------------------
    def draw_grads(self, step: int):
        for i in range(self.L):
            self.grads[i].copy_(draw_grad(self.w, i, step, self.device, scale=float(self.scales[i])))

    # ---- the path --------------------------------------------------------------------------------
    def hp(self, t: int) -> dict:
        w = self.w
        return dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, t=t, grad_dtype=self.grad_dtype,
                    inv_grad_scale=self.inv_scale, found_inf=self.found_inf, sr_seed=self.sr_seed)

    def step(self, t: int | None = None, stats: bool = False, new_bits=None, stream=None):
        """One optimizer step.  new_bits = (bits_m, bits_v) arrays switches widths inside the step."""
        self.t = self.t + 1 if t is None else t
        flags = stq.WITH_STATS if stats else 0
        if new_bits is None:
            self.handle.step(self.table(), flags=flags, stream=stream, **self.hp(self.t))
            return
        bm, bv = (np.asarray(a, dtype=np.uint8) for a in new_bits)
        new_states = []
        for i, n in enumerate(self.numels):
            if bm[i] == self.bits_m[i] and bv[i] == self.bits_v[i]:
                new_states.append(self.states[i])
            else:
                new_states.append(self._fresh_state(i, int(bm[i]), int(bv[i])))
        self.handle.step(self._make_table(self.states, new_states), flags=flags, stream=stream, **self.hp(self.t))
        self._adopt(new_states, bm, bv)

    def repack(self, new_bits, stream=None):
        """Width transition between steps."""
        bm, bv = (np.asarray(a, dtype=np.uint8) for a in new_bits)
        idx = [i for i in range(self.L) if bm[i] != self.bits_m[i] or bv[i] != self.bits_v[i]]
        if not idx:
            return
        new_states = list(self.states)
        rows = []
        for i in idx:
            new_states[i] = self._fresh_state(i, int(bm[i]), int(bv[i]))
            rows.append(stq.make_row(self.tab_numels[i], self.block, self.states[i], new_states[i], sr_id=i))
        self.handle.repack(stq.table(rows), stream=stream)
        self._adopt(new_states, bm, bv)

    def layer_stats(self, stream=None) -> np.ndarray:
        st = self.handle.layer_stats(self.L, stream=stream)
        if self.tile_padded:
            st[:, 3] = self.numels          # the element count of the real tensor (the sums have no share of the padding)
        return st

    def _fresh_state(self, i: int, bm: int, bv: int) -> stq.QState:
        """New buffers for the states whose width changes; unchanged states keep their buffers."""
        old = self.states[i]
        n = self.tab_numels[i]
        mc, ms = (old.m_codes, old.m_scales) if bm == old.bits_m else (
            stq.alloc_codes(n, bm, self.device), stq.alloc_scales(n, bm, self.block, self.device))
        vc, vs = (old.v_codes, old.v_scales) if bv == old.bits_v else (
            stq.alloc_codes(n, bv, self.device), stq.alloc_scales(n, bv, self.block, self.device, self.v_log))
        return stq.QState(mc, ms, bm, vc, vs, bv, self.v_log)

    def _adopt(self, new_states, bm, bv):
        torch.cuda.current_stream().synchronize()   # old buffers are released below
        self.states = new_states
        self.bits_m, self.bits_v = bm.copy(), bv.copy()
        self._tbl = None

    # ---- host mirror (for the host-buffer entry point) ------------------------------------------------
    def host_table(self, flat: bool = True):
        """Pinned host copies of everything a step reads and writes, and the table over them.

        flat: each kind of buffer (parameters, gradients, codes and scales of either state) lives in
        one pinned allocation, tensor after tensor at 256-byte aligned offsets, so that
        ``stq_step_host`` can move a chunk of tensors as one copy per kind.  Otherwise every state
        buffer is its own allocation.  Returns (table, host states, host parameters, host gradients)."""
        torch.cuda.synchronize(self.device)
        host_p = self.param_flat.cpu().pin_memory()
        host_g = self.grad_flat.cpu().pin_memory()

        def mirror(tensors):
            if not flat:
                return [t.cpu().pin_memory() for t in tensors]
            offs, total = [], 0
            for t in tensors:
                offs.append(total)
                total += _round_up(t.numel() * t.element_size(), 256)
            buf = torch.empty(max(total, 1), dtype=torch.uint8).pin_memory()
            out = []
            for t, o in zip(tensors, offs):
                v = buf[o:o + t.numel() * t.element_size()].view(t.dtype)
                v.copy_(t)
                out.append(v)
            return out

        mc, ms = mirror([s.m_codes for s in self.states]), mirror([s.m_scales for s in self.states])
        vc, vs = mirror([s.v_codes for s in self.states]), mirror([s.v_scales for s in self.states])
        states = [stq.QState(mc[i], ms[i], s.bits_m, vc[i], vs[i], s.bits_v, s.v_log) for i, s in enumerate(self.states)]
        rows = [stq.make_row(n, self.block, states[i], states[i], host_p[o:o + n], host_g[o:o + n], self.wd[i], sr_id=i)
                for i, (n, o) in enumerate(zip(self.tab_numels, self.offsets))]
        return stq.table(rows), states, host_p, host_g

    # ---- accounting ------------------------------------------------------------------------------
    def algorithmic_bytes(self) -> int:
        """Bytes one step must move (see the module-level function)."""
        return algorithmic_bytes(self.numels, self.bits_m, self.bits_v, self.block, self.w.grad_dtype,
                                 bool(self.w.lp_copy), 2 if self.w.v_log == "ts" else 1)

    def state_bytes(self) -> int:
        return int(sum(s.m_codes.numel() + s.v_codes.numel() + 4 * (s.m_scales.numel() + s.v_scales.numel())
                       for s in self.states))
