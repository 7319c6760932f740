"""Test-side glue: runs the CPU oracle next to the CUDA path on the same inputs and compares.

Only the tests (and the smoke check) import this; it is the one place where the oracle and the
product meet, and it contains no arithmetic of the method beyond the comparison itself.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2604_06836_b200 import stq

V_MODE = {"poly": O.LOG, "pl": O.LOG_PL, "sr": O.LOG_SR, "ts": O.LOG_TS}      # workload name -> oracle mode
from paper_2604_06836_b200.runner import Job


def to_np(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> numpy; bf16 comes back as its uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


class OracleJob:
    """The oracle's copy of a Job: same parameters, same widths, zero initial state."""

    def __init__(self, job: Job):
        self.w = job.w
        self.block = job.block
        self.numels = list(job.numels)
        self.theta = [to_np(p) for p in job.params]
        # largest magnitude each element (or one of its single-step changes) has had so far: rounding
        # differences are relative to the operands of the update, which may exceed the current value
        self.upd_mag = [np.abs(th) for th in self.theta]
        self.bits_m = job.bits_m.copy()
        self.bits_v = job.bits_v.copy()
        self.v_mode = V_MODE[job.w.v_log]
        self.sr_seed = job.sr_seed
        self.states = [O.new_state(n, self.block, int(bm), int(bv), self.v_mode)
                       for n, bm, bv in zip(self.numels, self.bits_m, self.bits_v)]
        self.wd = list(job.wd)

    def step(self, grads, t: int, want_stats=False, new_bits=None, decoupled_wd=True, fp16_grad=False,
             inv_grad_scale=1.0, found_inf=False):
        w = self.w
        stats = np.zeros((len(self.numels), 4))
        bm, bv = (self.bits_m, self.bits_v) if new_bits is None else (np.asarray(a, np.uint8) for a in new_bits)
        for i, g in enumerate(grads):
            before = self.theta[i].copy()
            self.states[i], s = O.step(self.theta[i], g, self.states[i], self.block, lr=w.lr, beta1=w.beta1,
                                       beta2=w.beta2, eps=w.eps, weight_decay=self.wd[i], t=t,
                                       bits_m_out=int(bm[i]), bits_v_out=int(bv[i]),
                                       decoupled_wd=decoupled_wd, want_stats=want_stats, fp16_grad=fp16_grad,
                                       inv_grad_scale=inv_grad_scale, found_inf=found_inf, v_mode=self.v_mode,
                                       sr_seed=self.sr_seed, tensor_index=i)
            self.upd_mag[i] = np.maximum(self.upd_mag[i], np.maximum(np.abs(self.theta[i] - before), np.abs(self.theta[i])))
            if want_stats:
                stats[i] = s
        self.bits_m, self.bits_v = np.array(bm, np.uint8), np.array(bv, np.uint8)
        return stats

    def repack(self, new_bits):
        bm, bv = (np.asarray(a, np.uint8) for a in new_bits)
        for i, n in enumerate(self.numels):
            st = self.states[i]
            if bm[i] != st.bits_m:
                st.m_codes, st.m_scales = O.repack(st.m_codes, st.m_scales, st.bits_m, int(bm[i]), n, self.block, O.LINEAR)
                st.bits_m = int(bm[i])
            if bv[i] != st.bits_v:
                st.v_codes, st.v_scales = O.repack(st.v_codes, st.v_scales, st.bits_v, int(bv[i]), n, self.block,
                                                   self.v_mode)
                st.bits_v = int(bv[i])
        self.bits_m, self.bits_v = bm.copy(), bv.copy()


def assert_states_equal(gs: stq.QState, os_: O.State, tag=""):
    """Packed codes and scales must agree byte for byte."""
    assert gs.bits_m == os_.bits_m and gs.bits_v == os_.bits_v, tag
    for name, g, o, bits in (("m", gs.m_codes, os_.m_codes, gs.bits_m), ("v", gs.v_codes, os_.v_codes, gs.bits_v)):
        g = to_np(g)
        assert g.size == o.size, (tag, name, g.size, o.size)
        if not (g == o).all():
            bad = np.flatnonzero(g != o)
            raise AssertionError(f"{tag}: {name} codes differ at {bad.size} bytes, first {bad[:8]} "
                                 f"gpu {g[bad[:8]]} oracle {o[bad[:8]]} (bits {bits})")
    for name, g, o, bits in (("m", gs.m_scales, os_.m_scales, gs.bits_m), ("v", gs.v_scales, os_.v_scales, gs.bits_v)):
        if bits == 32:
            continue
        g = to_np(g)
        if not (g.view(np.uint32) == o.view(np.uint32)).all():
            bad = np.flatnonzero(g.view(np.uint32) != o.view(np.uint32))
            raise AssertionError(f"{tag}: {name} scales differ at blocks {bad[:8]}: gpu {g[bad[:8]]} oracle {o[bad[:8]]}")


def assert_theta_close(g: torch.Tensor, o: np.ndarray, rel: float, tag="", upd: np.ndarray | None = None):
    """|a-b| <= rel * max(|b|, upd, 1e-3 * absmax(b)) element-wise, upd = largest magnitude the
    element or one of its single-step changes has had.

    The parameter is a difference of two fp32 terms (parameter, decay + update); where they nearly
    cancel, the error is relative to the terms, not to the small result, hence the upd leg."""
    g = to_np(g).astype(np.float64)
    o = o.astype(np.float64)
    floor = 1e-3 * np.abs(o).max() if o.size else 0.0
    mag = np.maximum(np.abs(o), floor)
    if upd is not None:
        mag = np.maximum(mag, upd.astype(np.float64))
    lim = rel * mag
    err = np.abs(g - o)
    if not (err <= lim).all():
        k = int(np.argmax(err / np.maximum(lim, 1e-300)))
        raise AssertionError(f"{tag}: theta differs: idx {k} gpu {g[k]!r} oracle {o[k]!r} err {err[k]:.3e} lim {lim[k]:.3e}")


def assert_stats_close(g: np.ndarray, o: np.ndarray, tag=""):
    assert g.shape == o.shape
    # sum g cancels, so it is held to the scale of sum |g|
    assert (np.abs(g[:, 0] - o[:, 0]) <= 2e-6 * np.maximum(o[:, 1], 1e-300)).all(), (tag, g[:, 0], o[:, 0])
    np.testing.assert_allclose(g[:, 1], o[:, 1], rtol=2e-6, err_msg=tag)
    np.testing.assert_allclose(g[:, 2], o[:, 2], rtol=2e-6, err_msg=tag)
    assert (g[:, 3] == o[:, 3]).all()


def compare_job(job: Job, oj: OracleJob, rel: float, tag=""):
    job.handle.device_status()      # synchronises; raises if a kernel gave up on a bounded wait
    for i in range(job.L):
        assert_states_equal(job.states[i], oj.states[i], f"{tag} tensor {i} ({job.w.shapes[i][0]})")
        assert_theta_close(job.params[i], oj.theta[i], rel, f"{tag} tensor {i} ({job.w.shapes[i][0]})",
                           upd=oj.upd_mag[i])


class SampledOracle:
    """Oracle on a sample of quantization blocks of a full-size Job.

    Blocks are independent given (theta, grad, stored state), so a few blocks per tensor, gathered
    into a small tensor (the ragged last block, if any, goes last), can be stepped by the oracle one
    by one and compared with the same blocks of the GPU buffers."""

    def __init__(self, job: Job, per_tensor: int = 6, seed: int = 0):
        self.job = job
        self.block = job.block
        rng = np.random.RandomState(seed)
        self.sel, self.n_mini = [], []
        for n in job.numels:
            nb_full = n // self.block
            tail = n - nb_full * self.block
            pick = set()
            if nb_full:
                pick.update([0, nb_full - 1])
                # blocks on either side of tile boundaries (4096 elements) and random ones
                for b in (4096 // self.block - 1, 4096 // self.block):
                    if b < nb_full:
                        pick.add(b)
                pick.update(rng.randint(0, nb_full, size=per_tensor).tolist())
            blocks = sorted(pick)
            self.sel.append((np.array(blocks, dtype=np.int64), tail, nb_full))
            self.n_mini.append(len(blocks) * self.block + tail)
        self.theta = [self._gather_elems(p, i) for i, p in enumerate(job.params)]
        self.v_mode = V_MODE[job.w.v_log]
        assert self.v_mode != O.LOG_SR, "the random words belong to element positions: sample-free checks only"
        self.states = [O.new_state(self.n_mini[i], self.block, int(job.bits_m[i]), int(job.bits_v[i]), self.v_mode)
                       for i in range(job.L)]
        self.mag = [np.abs(t) for t in self.theta]
        self.stepped = False      # the working copy exists only after the first step

    def _elem_index(self, i: int) -> torch.Tensor:
        blocks, tail, nb_full = self.sel[i]
        idx = (blocks[:, None] * self.block + np.arange(self.block)[None, :]).ravel()
        if tail:
            idx = np.concatenate([idx, nb_full * self.block + np.arange(tail)])
        return torch.from_numpy(idx).to(self.job.device)

    def _gather_elems(self, t: torch.Tensor, i: int) -> np.ndarray:
        return to_np(t[self._elem_index(i)])

    def _gather_codes(self, codes: torch.Tensor, bits: int, i: int) -> np.ndarray:
        blocks, tail, nb_full = self.sel[i]
        bb = self.block * bits // 8
        idx = (blocks[:, None] * bb + np.arange(bb)[None, :]).ravel()
        if tail:
            idx = np.concatenate([idx, nb_full * bb + np.arange((tail * bits + 7) // 8)])
        got = to_np(codes[torch.from_numpy(idx).to(codes.device)])
        out = np.zeros(O.codes_bytes(self.n_mini[i], bits), dtype=np.uint8)
        out[:got.size] = got
        return out

    def _gather_scales(self, scales: torch.Tensor, i: int) -> np.ndarray:
        blocks, tail, nb_full = self.sel[i]
        idx = np.concatenate([blocks, [nb_full]]) if tail else blocks
        return to_np(scales[torch.from_numpy(idx).to(scales.device)])

    def step(self, t: int, new_bits=None):
        """Oracle step on the sample, with the gradients currently held by the job.  new_bits =
        (bits_m, bits_v) arrays switches widths inside the step."""
        w = self.job.w
        self.stepped = True
        for i in range(self.job.L):
            if self.n_mini[i] == 0:
                continue
            g = self._gather_elems(self.job.grads[i], i)
            before = self.theta[i].copy()
            bm = None if new_bits is None else int(new_bits[0][i])
            bv = None if new_bits is None else int(new_bits[1][i])
            amp = dict(fp16_grad=True, inv_grad_scale=1.0 / w.loss_scale) if w.grad_dtype == "fp16" else {}
            self.states[i], _ = O.step(self.theta[i], g, self.states[i], self.block, lr=w.lr, beta1=w.beta1,
                                       beta2=w.beta2, eps=w.eps, weight_decay=self.job.wd[i], t=t,
                                       bits_m_out=bm, bits_v_out=bv, v_mode=self.v_mode, **amp)
            self.mag[i] = np.maximum(self.mag[i], np.maximum(np.abs(self.theta[i]), np.abs(self.theta[i] - before)))

    def repack(self, new_bits):
        """Width transition between steps on the sampled blocks."""
        for i in range(self.job.L):
            st, n = self.states[i], self.n_mini[i]
            if n == 0:
                continue
            bm, bv = int(new_bits[0][i]), int(new_bits[1][i])
            if bm != st.bits_m:
                st.m_codes, st.m_scales = O.repack(st.m_codes, st.m_scales, st.bits_m, bm, n, self.block, O.LINEAR)
                st.bits_m = bm
            if bv != st.bits_v:
                st.v_codes, st.v_scales = O.repack(st.v_codes, st.v_scales, st.bits_v, bv, n, self.block, self.v_mode)
                st.bits_v = bv

    def compare(self, rel: float, tag=""):
        job = self.job
        job.handle.device_status()
        for i in range(job.L):
            if self.n_mini[i] == 0:
                continue
            gs, os_ = job.states[i], self.states[i]
            name = f"{tag} tensor {i} ({job.w.shapes[i][0]}, bits {gs.bits_m}/{gs.bits_v})"
            assert (self._gather_codes(gs.m_codes, gs.bits_m, i) == os_.m_codes).all(), name + " m codes"
            assert (self._gather_codes(gs.v_codes, gs.bits_v, i) == os_.v_codes).all(), name + " v codes"
            assert (self._gather_scales(gs.m_scales, i).view(np.uint32) == os_.m_scales.view(np.uint32)).all(), name
            assert (self._gather_scales(gs.v_scales, i).view(np.uint32) == os_.v_scales.view(np.uint32)).all(), name
            g = self._gather_elems(job.params[i], i).astype(np.float64)
            o = self.theta[i].astype(np.float64)
            lim = rel * np.maximum(self.mag[i].astype(np.float64), 1e-3 * np.abs(o).max())
            assert (np.abs(g - o) <= lim).all(), name + f" theta: max err {np.abs(g - o).max():.3e}"
            if job.w.lp_copy and self.stepped:   # the working copy is the kernel's own fp32 result, rounded to nearest even
                idx = self._elem_index(i)
                lp = job.params_lp[i]
                assert torch.equal(lp[idx], job.params[i][idx].to(lp.dtype)), name + " working copy"


class FullOracle:
    """Oracle on EVERY element of a full-size Job.

    Quantization blocks are independent given their inputs, so each tensor is cut into ranges that start
    on block boundaries and the ranges are stepped by a pool of host threads (the oracle's C code runs
    outside the interpreter lock).  The oracle's own state starts from its own zero initialisation and is
    never fed from the CUDA path; only the seeded parameter and gradient draws are shared.  The comparison
    covers whole buffers (every code byte, every scale, every parameter) and runs on the device to keep
    the test short."""

    def __init__(self, job: Job, range_elems: int = 1 << 21, threads: int | None = None):
        import os
        from concurrent.futures import ThreadPoolExecutor
        self.job, self.w, self.block = job, job.w, job.block
        assert range_elems % 1024 == 0
        self.range_elems = range_elems
        self.pool = ThreadPoolExecutor(max_workers=threads or os.cpu_count() or 4)
        self.theta = [to_np(p) for p in job.params]
        self.v_mode = V_MODE[job.w.v_log]
        self.states = [O.new_state(n, self.block, int(bm), int(bv), self.v_mode)
                       for n, bm, bv in zip(job.numels, job.bits_m, job.bits_v)]
        self.mag = [p.abs() for p in job.params]          # device: largest magnitude an element or its step has had
        self.theta_dev = [p.clone() for p in job.params]  # device copy of the oracle's parameters (same bits at the start)

    def _ranges(self):
        for i, n in enumerate(self.job.numels):
            for e0 in range(0, n, self.range_elems):
                yield i, e0, min(n, e0 + self.range_elems)

    def step(self, t: int, new_bits=None, want_stats: bool = False) -> np.ndarray:
        """One oracle step on the gradients the job currently holds.  Returns [L, 4] sums (zeros unless asked)."""
        job, w = self.job, self.w

        def host(t):        # one copy to the host; the array keeps the host tensor alive
            t = t.detach().cpu()
            return t.view(torch.int16).numpy().view(np.uint16) if t.dtype in (torch.bfloat16, torch.float16) else t.numpy()
        grads = [host(g) for g in job.grads]
        out = []
        for i, n in enumerate(job.numels):
            bm = self.states[i].bits_m if new_bits is None else int(new_bits[0][i])
            bv = self.states[i].bits_v if new_bits is None else int(new_bits[1][i])
            mc, ms = O.alloc_state(n, bm, self.block)
            vc, vs = O.alloc_state(n, bv, self.block, self.v_mode)
            out.append(O.State(mc, ms, bm, vc, vs, bv))
        amp = dict(fp16_grad=True, inv_grad_scale=1.0 / w.loss_scale) if w.grad_dtype == "fp16" else {}
        tasks = list(self._ranges())
        part = np.zeros((len(tasks), 4))

        def run(k):
            i, e0, e1 = tasks[k]
            O.step_range(self.theta[i], grads[i], e0, e1, self.block, self.states[i], out[i], lr=w.lr, beta1=w.beta1,
                         beta2=w.beta2, eps=w.eps, weight_decay=job.wd[i], t=t, v_mode=self.v_mode,
                         stats=part[k] if want_stats else None, sr_seed=job.sr_seed, tensor_index=i, **amp)

        list(self.pool.map(run, range(len(tasks))))
        self.states = out
        for i in range(job.L):
            now = torch.from_numpy(self.theta[i]).to(job.device)
            self.mag[i] = torch.maximum(self.mag[i], torch.maximum(now.abs(), (now - self.theta_dev[i]).abs()))
            self.theta_dev[i] = now
        stats = np.zeros((job.L, 4))
        for k, (i, _, _) in enumerate(tasks):
            stats[i] += part[k]
        return stats

    def repack(self, new_bits):
        def run(i):
            st, n = self.states[i], self.job.numels[i]
            bm, bv = int(new_bits[0][i]), int(new_bits[1][i])
            if bm != st.bits_m:
                st.m_codes, st.m_scales = O.repack(st.m_codes, st.m_scales, st.bits_m, bm, n, self.block, O.LINEAR)
                st.bits_m = bm
            if bv != st.bits_v:
                st.v_codes, st.v_scales = O.repack(st.v_codes, st.v_scales, st.bits_v, bv, n, self.block, self.v_mode)
                st.bits_v = bv
        list(self.pool.map(run, range(self.job.L)))

    def compare(self, rel: float, tag=""):
        """Whole buffers: codes and scales byte for byte, parameters to rel * max(|b|, largest magnitude the
        element or its step has had, 1e-3 * absmax of the tensor)."""
        job = self.job
        job.handle.device_status()
        dev = job.device
        for i in range(job.L):
            gs, os_ = job.states[i], self.states[i]
            name = f"{tag} tensor {i} ({job.w.shapes[i][0]}, bits {gs.bits_m}/{gs.bits_v})"
            assert gs.bits_m == os_.bits_m and gs.bits_v == os_.bits_v, name
            padded = getattr(job, "tile_padded", False)
            n = job.numels[i]
            for what, g, o, b in (("m codes", gs.m_codes, os_.m_codes, gs.bits_m), ("v codes", gs.v_codes, os_.v_codes, gs.bits_v)):
                o_d = torch.from_numpy(o).to(dev)
                if padded:
                    # the job's buffers run on into the zero padding: the codes of the real elements are a prefix of
                    # the bit stream (whole bytes, then the low bits of one more)
                    whole, rest = (n * b) // 8, (n * b) % 8
                    g, o_d = g.view(torch.uint8)[:whole + (rest > 0)].clone(), o_d.view(torch.uint8)[:whole + (rest > 0)].clone()
                    if rest:
                        g[-1] &= (1 << rest) - 1
                        o_d[-1] &= (1 << rest) - 1
                if not torch.equal(g, o_d):
                    bad = torch.nonzero(g != o_d).flatten()[:8].tolist()
                    raise AssertionError(f"{name}: {what} differ at bytes {bad}")
            for what, g, o, b in (("m scales", gs.m_scales, os_.m_scales, gs.bits_m),
                                  ("v scales", gs.v_scales, os_.v_scales, gs.bits_v)):
                if b == 32:
                    continue
                o_d = torch.from_numpy(o).to(dev)
                if padded:
                    g = g[:o_d.numel()]                      # the blocks that hold real elements
                if not torch.equal(g.view(torch.int32), o_d.view(torch.int32)):
                    bad = torch.nonzero(g.view(torch.int32) != o_d.view(torch.int32)).flatten()[:8].tolist()
                    raise AssertionError(f"{name}: {what} differ at blocks {bad}")
            o = self.theta_dev[i].double()
            g = job.params[i].double()
            lim = rel * torch.maximum(self.mag[i].double(), 1e-3 * o.abs().max())
            err = (g - o).abs()
            if not bool((err <= lim).all()):
                k = int(torch.argmax(err / lim.clamp_min(1e-300)))
                raise AssertionError(f"{name}: theta differs at {k}: gpu {float(g[k])!r} oracle {float(o[k])!r} "
                                     f"err {float(err[k]):.3e} lim {float(lim[k]):.3e}")
