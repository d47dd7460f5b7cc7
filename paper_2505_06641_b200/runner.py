"""Convenience driver around the C ABI: keeps a workload's request arrays on the device and runs the path.

Only marshalling and buffer management live here; all arithmetic runs in the CUDA library.  PyTorch is
used for device memory and the CUDA stream.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import api


@dataclass
class Result:
    acc: Optional[np.ndarray]      # [n, Mmax] float32
    v: Optional[np.ndarray]        # [n] float32
    reqs: np.ndarray               # [n] api.REQ_DTYPE
    rounds: np.ndarray             # [I, cap] api.ROUND_DTYPE
    n_rounds: np.ndarray           # [I] int32
    t_end_ns: np.ndarray           # [I] int64
    loaded_end: np.ndarray         # [I] int32
    stats: dict


def _bits_tensor(a: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor with the same bits."""
    return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)


class Session:
    """One library context bound to a workload's profiles; requests live in device tensors."""

    def __init__(self, w, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.w = w
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.stream = torch.cuda.current_stream(self.device)
        self.ctx = api.sp_create(device, self.stream.cuda_stream)
        api.sp_load_profiles(self.ctx, w)
        api.sp_set_options(self.ctx, trace_mode=bool(w.trace_mode))
        self.n = int(w.app.shape[0])
        self.mmax = int(np.max(w.models_per_app))
        self.dev = None

    def close(self):
        if self.ctx:
            api.sp_destroy(self.ctx)
            self.ctx = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def upload(self):
        """Copies the request arrays to the device (outside any timed region)."""
        w, d = self.w, self.device
        feats = _bits_tensor(w.feats, d) if int(w.feat_dtype) == api.SP_BF16 else torch.from_numpy(w.feats).to(d)
        self.dev = dict(
            feats=feats.contiguous(), app=torch.from_numpy(np.ascontiguousarray(w.app, dtype=np.int32)).to(d),
            arrival=torch.from_numpy(np.ascontiguousarray(w.arrival_ns, dtype=np.int64)).to(d),
            deadline=torch.from_numpy(np.ascontiguousarray(w.deadline_ns, dtype=np.int64)).to(d),
            instance=(torch.from_numpy(np.ascontiguousarray(w.instance, dtype=np.int32)).to(d)
                      if int(w.n_instances) > 1 else None),
            t0=torch.from_numpy(np.ascontiguousarray(w.t0_ns, dtype=np.int64)).to(d),
            l0=torch.full((int(w.n_instances),), -1, dtype=torch.int32, device=d))
        return self.dev

    def alloc_outputs(self, cap: int):
        ni, d = int(self.w.n_instances), self.device
        self.cap = int(cap)
        self.rounds = torch.zeros((ni, self.cap, api.ROUND_DTYPE.itemsize), dtype=torch.uint8, device=d)
        self.n_done = torch.zeros(ni, dtype=torch.int32, device=d)
        self.recs = torch.zeros((max(self.n, 1), api.REQ_DTYPE.itemsize), dtype=torch.uint8, device=d)

    def score(self, acc_out=None):
        dv = self.dev
        api.sp_reset(self.ctx)
        api.sp_set_clocks(self.ctx, dv["t0"], dv["l0"])      # every run starts at t0 with no model resident
        api.sp_score(self.ctx, self.n, dv["feats"], dv["app"], dv["arrival"], dv["deadline"], dv["instance"], acc_out)

    def schedule(self, max_rounds: int):
        api.sp_schedule_round(self.ctx, max_rounds, self.rounds, self.cap, self.n_done)

    def run(self, max_rounds: Optional[int] = None, cap: Optional[int] = None, loaded0: Optional[np.ndarray] = None,
            want_scores: bool = True) -> Result:
        """Scores every request and runs the rounds; returns everything on the host."""
        w, ni = self.w, int(self.w.n_instances)
        if self.dev is None:
            self.upload()
        per_inst = int(np.max(np.bincount(np.asarray(w.instance), minlength=ni))) if self.n else 0
        if max_rounds is None:
            max_rounds = per_inst + 1
        if cap is None:
            cap = max(1, min(max_rounds, per_inst))
        self.alloc_outputs(cap)
        self.score()
        if loaded0 is not None:
            api.sp_set_clocks(self.ctx, None, torch.from_numpy(np.ascontiguousarray(loaded0, dtype=np.int32)).to(self.device))
        self.schedule(max_rounds)
        acc = v = None
        if want_scores and self.n:
            acc_t = torch.empty((self.n, self.mmax), dtype=torch.float32, device=self.device)
            v_t = torch.empty(self.n, dtype=torch.float32, device=self.device)
            api.sp_get_scores(self.ctx, 0, self.n, acc_t, v_t)
        if self.n:
            api.sp_get_requests(self.ctx, 0, self.n, self.recs)
        t_end = torch.empty(ni, dtype=torch.int64, device=self.device)
        l_end = torch.empty(ni, dtype=torch.int32, device=self.device)
        api.sp_get_clocks(self.ctx, t_end, l_end)
        api.sp_check(self.ctx)
        if want_scores and self.n:
            acc, v = acc_t.cpu().numpy(), v_t.cpu().numpy()
        reqs = self.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:self.n]
        rounds = self.rounds.cpu().numpy().reshape(ni, -1).view(api.ROUND_DTYPE)
        return Result(acc, v, reqs, rounds, self.n_done.cpu().numpy(), t_end.cpu().numpy(), l_end.cpu().numpy(),
                      api.sp_get_stats(self.ctx))
