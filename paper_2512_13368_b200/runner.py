"""Device-buffer plumbing around the C ABI: upload a workload, allocate outputs and the
workspace with PyTorch, call the library, hand results back.  No arithmetic of the method
happens here."""
from __future__ import annotations

import os

import numpy as np
import torch

from . import binding
from .workloads import Workload

_TORCH_DTYPE = {"fp32": torch.float32, "bf16": torch.bfloat16}


class DeviceProblem:
    """All device buffers of one forward + backward call for a workload."""

    def __init__(self, w: Workload, device="cuda:0", sm_scale=0.0, training=True):
        self.w = w
        self.device = torch.device(device)
        dt = _TORCH_DTYPE[w.dtype]
        self.dt = dt
        up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.device).to(dt)  # noqa: E731
        self.q, self.k, self.v, self.dout = up(w.q), up(w.k), up(w.v), up(w.dout)
        self.gate = torch.from_numpy(np.ascontiguousarray(w.gate, dtype=np.float32)).to(self.device)
        self.seq_lens = None
        if w.seq_lens is not None:
            self.seq_lens = torch.from_numpy(w.seq_lens.astype(np.int32)).to(self.device)
        self.phi = None   # logits of the learnable block summary, kept alive here (the params hold its address)
        if getattr(w, "phi_logits", None) is not None:
            self.phi = torch.from_numpy(np.ascontiguousarray(w.phi_logits, dtype=np.float32)).to(self.device)
        self.params = binding.make_params(w.B, w.H, w.L, w.D, w.block, w.topk, w.window, w.dtype,
                                          sm_scale=sm_scale, stis_mode=w.stis_mode,
                                          stis_block=w.stis_block, cmp_block=w.cmp_block,
                                          cmp_stride=w.cmp_stride, kv_heads=w.kv_heads or w.H,
                                          select_mode=w.per_query, phi_logits=self.phi,
                                          gate_mode=getattr(w, "gate_mode", 0), causal=getattr(w, "causal", 1),
                                          rope_theta=getattr(w, "rope_theta", 0.0))
        # the backward of a step follows its training forward on the same workspace: it reuses the
        # tile lists that forward left there
        self.params_bwd = binding.blossom_params.from_buffer_copy(self.params)
        self.params_bwd.reuse_tile_lists = 1
        self.alloc_outputs(training)

    def alloc_outputs(self, training=True):
        w, dev = self.w, self.device
        shape = (w.B, w.H, w.L, w.D)
        e = lambda: torch.empty(shape, dtype=self.dt, device=dev)  # noqa: E731
        hkv = w.kv_heads or w.H   # k, v, dk, dv and the selection are per key/value head
        ekv = lambda: torch.empty((w.B, hkv, w.L, w.D), dtype=self.dt, device=dev)  # noqa: E731
        rows = w.L if w.per_query else w.n_blocks   # one index row per position or per query block
        self.idx = torch.empty((w.B, hkv, rows, w.topk), dtype=torch.int32, device=dev)
        self.out = e()
        self.out_lt = e() if training else None
        self.out_st = e() if training else None
        self.lse = torch.empty((2, w.B, w.H, w.L), dtype=torch.float32, device=dev) if training else None
        self.dq, self.dk, self.dv = (e(), ekv(), ekv()) if training else (None, None, None)
        self.dgate = torch.empty(tuple(w.gate.shape), dtype=torch.float32, device=dev)
        nbytes = binding.blossom_workspace_bytes(self.params)
        if nbytes == 0:
            raise binding.BlossomError(binding.BLOSSOM_ERR_UNSUPPORTED, "blossom_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        if os.environ.get("BLOSSOM_POISON_BUFFERS", "0") not in ("", "0"):
            # debugging aid: every output and the workspace start as 0xFF bytes (NaN in bf16 and
            # fp32, -1 as int32), so that a read of memory nobody has written shows in the results
            # instead of finding the still-correct leftovers of an earlier, identical run
            for t in (self.idx, self.out, self.out_lt, self.out_st, self.lse, self.dq, self.dk, self.dv,
                      self.dgate, self.workspace):
                if t is not None:
                    t.view(torch.uint8).fill_(0xFF)

    # -- calls ---------------------------------------------------------------------------
    def select(self, stream=None):
        binding.blossom_select_blocks(self.params, self.q, self.k, self.seq_lens, self.idx,
                                      self.workspace, stream=stream)

    def forward(self, idx_is_input=False, stream=None):
        binding.blossom_attn_fwd(self.params, self.q, self.k, self.v, self.gate, self.seq_lens,
                                 self.idx, int(idx_is_input), self.out, self.out_lt, self.out_st,
                                 self.lse, self.workspace, stream=stream)

    def backward(self, stream=None, reuse_tile_lists=True):
        binding.blossom_attn_bwd(self.params_bwd if reuse_tile_lists else self.params, self.q, self.k, self.v, self.gate, self.seq_lens,
                                 self.idx, self.out_lt, self.out_st, self.lse, self.dout, self.dq,
                                 self.dk, self.dv, self.dgate, self.workspace, stream=stream)

    def step(self, stream=None):
        """One pass of the whole hot path: selection + forward + backward."""
        self.forward(False, stream)
        self.backward(stream)

    # -- results -------------------------------------------------------------------------
    def results(self) -> dict:
        torch.cuda.synchronize(self.device)
        f = lambda t: None if t is None else t.float().cpu().numpy()  # noqa: E731
        return {"idx": self.idx.cpu().numpy(), "out": f(self.out), "out_lt": f(self.out_lt),
                "out_st": f(self.out_st), "lse": f(self.lse), "dq": f(self.dq), "dk": f(self.dk),
                "dv": f(self.dv), "dgate": f(self.dgate)}


class HostPipeline:
    """Steps whose inputs and results live in pinned host memory.

    `slots` device problems take turns: while one computes, the next one's inputs are uploaded
    and the previous one's results are downloaded, on three streams ordered by events (PCIe
    carries both directions at once).  Every byte of every step crosses the bus; only the
    waiting is taken out.  The host buffers of a submitted step must stay untouched until
    `drain()` (or until `slots` further steps have been submitted).
    """

    IN = ("q", "k", "v", "dout", "gate")
    OUT = ("out", "dq", "dk", "dv", "dgate")

    def __init__(self, w: Workload, slots: int = 2, device="cuda:0", sm_scale=0.0):
        self.device = torch.device(device)
        self.slots = [DeviceProblem(w, device, sm_scale) for _ in range(slots)]
        mk = lambda: [torch.cuda.Event() for _ in range(slots)]  # noqa: E731
        self.uploaded, self.computed, self.downloaded = mk(), mk(), mk()
        self.s_up, self.s_run, self.s_down = (torch.cuda.Stream(self.device) for _ in range(3))
        self.n = 0

    def pinned_inputs(self) -> dict:
        p = self.slots[0]
        d = {k: getattr(p, k).detach().cpu().pin_memory() for k in self.IN}
        if p.seq_lens is not None:
            d["seq_lens"] = p.seq_lens.cpu().pin_memory()
        return d

    def pinned_outputs(self) -> dict:
        p = self.slots[0]
        return {k: torch.empty(getattr(p, k).shape, dtype=getattr(p, k).dtype).pin_memory() for k in self.OUT}

    def submit(self, h_in: dict, h_out: dict):
        i = self.n % len(self.slots)
        p = self.slots[i]
        used = self.n >= len(self.slots)
        with torch.cuda.stream(self.s_up):
            if used:
                self.s_up.wait_event(self.computed[i])      # the slot's last step has read its inputs
            for k, h in h_in.items():
                getattr(p, k).copy_(h, non_blocking=True)
            self.uploaded[i].record(self.s_up)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(self.uploaded[i])
            if used:
                self.s_run.wait_event(self.downloaded[i])   # and its results have left the device
            p.step()
            self.computed[i].record(self.s_run)
        with torch.cuda.stream(self.s_down):
            self.s_down.wait_event(self.computed[i])
            for k, h in h_out.items():
                h.copy_(getattr(p, k), non_blocking=True)
            self.downloaded[i].record(self.s_down)
        self.n += 1

    def fence(self, stream=None):
        """Makes `stream` (default: the current one) wait for everything submitted so far, and the
        pipeline's streams wait for what `stream` has done."""
        cur = stream or torch.cuda.current_stream(self.device)
        e = torch.cuda.Event()
        e.record(cur)
        for s in (self.s_up, self.s_run, self.s_down):
            s.wait_event(e)
            d = torch.cuda.Event()
            d.record(s)
            cur.wait_event(d)

    def drain(self):
        for s in (self.s_up, self.s_run, self.s_down):
            s.synchronize()
