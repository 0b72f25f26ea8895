"""Allocation helpers around the C ABI: put a synthetic workload on the device, run the backward,
bring the gradients back.  PyTorch is used for device memory and streams only."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

from . import binding
from .synth import Workload


def _io_dtype(wl: Workload):
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def desc_for(wl: Workload) -> binding.gdn_desc:
    return binding.make_desc(B=wl.B, T=wl.T, H=wl.H, d_k=wl.d_k, d_v=wl.d_v, N=wl.N, dtype=wl.dtype,
                             scale=wl.scale, delta_rule=wl.delta_rule, chunk=wl.chunk)


@dataclass
class DeviceBuffers:
    desc: binding.gdn_desc
    inputs: Dict[str, Optional[torch.Tensor]]
    outputs: Dict[str, Optional[torch.Tensor]]
    workspace: torch.Tensor


def host_inputs(wl: Workload, pin: bool = False) -> Dict[str, Optional[torch.Tensor]]:
    """Host tensors in the I/O dtype (bf16 values are already exactly representable)."""
    io = _io_dtype(wl)
    def t(a, dt):
        if a is None:
            return None
        x = torch.from_numpy(np.ascontiguousarray(a)).to(dt)
        return x.pin_memory() if pin else x
    return dict(q=t(wl.q, io), k=t(wl.k, io), v=t(wl.v, io), dO=t(wl.dO, io), g=t(wl.g, torch.float32),
                beta=t(wl.beta, torch.float32), h0=t(wl.h0, torch.float32), dhT=t(wl.dhT, torch.float32),
                cu_seqlens=t(wl.cu_seqlens, torch.int32) if wl.varlen else None)


def to_device(wl: Workload, device="cuda:0", want_o: bool = False) -> DeviceBuffers:
    io = _io_dtype(wl)
    dev = torch.device(device)
    hin = host_inputs(wl)
    inputs = {k: (None if v is None else v.to(dev)) for k, v in hin.items()}
    Tt, H, N = wl.T_total, wl.H, wl.N
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
    outputs = dict(dq=z((Tt, H, wl.d_k), io), dk=z((Tt, H, wl.d_k), io), dv=z((Tt, H, wl.d_v), io),
                   dg=z((Tt, H), torch.float32), dbeta=z((Tt, H), torch.float32) if wl.delta_rule else None,
                   dh0=z((N, H, wl.d_k, wl.d_v), torch.float32),
                   o=z((Tt, H, wl.d_v), io) if want_o else None,
                   hT=z((N, H, wl.d_k, wl.d_v), torch.float32) if want_o else None)
    desc = desc_for(wl)
    _, bwd_bytes = binding.gdn_workspace_bytes(desc)
    ws = torch.empty(bwd_bytes, dtype=torch.uint8, device=dev)
    return DeviceBuffers(desc=desc, inputs=inputs, outputs=outputs, workspace=ws)


def run_fwd(buf: DeviceBuffers, stream=None) -> None:
    i, o = buf.inputs, buf.outputs
    binding.gdn_fwd_recompute(buf.desc, i["q"], i["k"], i["v"], i["g"], i["beta"], i["h0"], i["cu_seqlens"],
                              o["o"], o["hT"], buf.workspace, stream=stream)


def run_bwd(buf: DeviceBuffers, fresh: int = 0, stream=None) -> None:
    i, o = buf.inputs, buf.outputs
    binding.gdn_bwd(buf.desc, i["q"], i["k"], i["v"], i["g"], i["beta"], i["h0"], i["dO"], i["dhT"],
                    i["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["dbeta"], o["dh0"], buf.workspace,
                    workspace_is_fresh_from_fwd=fresh, stream=stream)


def fetch(buf: DeviceBuffers) -> Dict[str, np.ndarray]:
    """Synchronise, check the device status word, return outputs as float64 numpy arrays."""
    st = binding.gdn_last_device_status(buf.workspace)
    if st != binding.GDN_OK:
        raise binding.GdnError(st, "device status")
    return {k: v.detach().to(torch.float64).cpu().numpy() for k, v in buf.outputs.items() if v is not None}


def backward(wl: Workload, device="cuda:0") -> Dict[str, np.ndarray]:
    """One-shot convenience: upload, gdn_bwd, download."""
    buf = to_device(wl, device)
    run_bwd(buf)
    return fetch(buf)


class HostBackward:
    """`gdn_bwd` for callers whose tensors live in host memory.

    Sequences are independent, so a fixed-length batch is cut into pieces of whole sequences; the upload of a piece,
    the kernels of the previous piece and the download of the one before run on three streams and overlap (PCIe is
    full duplex).  Packed variable-length input and single-sequence batches run as one piece.  Host tensors are
    pinned; `inputs` and `outputs` are the host-side views a caller fills and reads.
    """

    def __init__(self, wl: Workload, device="cuda:0", pieces: Optional[int] = None):
        self.dev = torch.device(device)
        self.wl = wl
        if wl.varlen or wl.B == 1:
            pieces = 1
        elif pieces is None:
            pieces = wl.B
        if wl.B % pieces:
            raise ValueError("pieces must divide the batch")
        self.pieces = pieces
        self.inputs = host_inputs(wl, pin=True)
        io = _io_dtype(wl)
        Tt, H, N = wl.T_total, wl.H, wl.N
        hz = lambda shape, dt: torch.zeros(shape, dtype=dt).pin_memory()
        self.outputs = dict(dq=hz((Tt, H, wl.d_k), io), dk=hz((Tt, H, wl.d_k), io), dv=hz((Tt, H, wl.d_v), io),
                            dg=hz((Tt, H), torch.float32), dbeta=hz((Tt, H), torch.float32) if wl.delta_rule else None,
                            dh0=hz((N, H, wl.d_k, wl.d_v), torch.float32))
        bp = wl.B // pieces                         # sequences per piece (packed input: one piece, all of it)
        rows = Tt if wl.varlen else bp * wl.T       # token rows per piece
        seqs = N if wl.varlen else bp               # sequences (state tensors) per piece
        self._rows, self._seqs = rows, seqs
        self._desc = binding.make_desc(B=bp, T=wl.T, H=H, d_k=wl.d_k, d_v=wl.d_v, N=seqs, dtype=wl.dtype,
                                       scale=wl.scale, delta_rule=wl.delta_rule, chunk=wl.chunk)
        _, ws_bytes = binding.gdn_workspace_bytes(self._desc)

        def device_like(name: str, host: Optional[torch.Tensor]) -> Optional[torch.Tensor]:
            if host is None:
                return None
            lead = host.shape[0] if name == "cu_seqlens" else (seqs if name in ("h0", "dhT", "dh0") else rows)
            return torch.zeros((lead,) + tuple(host.shape[1:]), dtype=host.dtype, device=self.dev)

        self._slots = []
        for _ in range(pieces):
            self._slots.append(dict(inp={k: device_like(k, v) for k, v in self.inputs.items()},
                                    out={k: device_like(k, v) for k, v in self.outputs.items()},
                                    ws=torch.empty(ws_bytes, dtype=torch.uint8, device=self.dev),
                                    ev_in=torch.cuda.Event(), ev_c=torch.cuda.Event()))
        self._s_in, self._s_c, self._s_out = (torch.cuda.Stream(self.dev) for _ in range(3))
        self.h2d_bytes = sum(v.numel() * v.element_size() for v in self.inputs.values() if v is not None)
        self.d2h_bytes = sum(v.numel() * v.element_size() for v in self.outputs.values() if v is not None)

    def _host_slice(self, t: torch.Tensor, name: str, i: int) -> torch.Tensor:
        if name == "cu_seqlens":
            return t
        n = self._seqs if name in ("h0", "dhT", "dh0") else self._rows
        return t[i * n:(i + 1) * n]

    def step(self) -> None:
        """Enqueue one backward of the whole batch, ordered after the caller's current stream; the current stream
        waits for the last download, so an event recorded on it afterwards marks the end of the step."""
        cur = torch.cuda.current_stream(self.dev)
        for s in (self._s_in, self._s_c, self._s_out):
            s.wait_stream(cur)
        for i, sl in enumerate(self._slots):
            with torch.cuda.stream(self._s_in):
                for k, v in self.inputs.items():
                    if v is not None:
                        sl["inp"][k].copy_(self._host_slice(v, k, i), non_blocking=True)
                sl["ev_in"].record(self._s_in)
            with torch.cuda.stream(self._s_c):
                self._s_c.wait_event(sl["ev_in"])
                a, o = sl["inp"], sl["out"]
                binding.gdn_bwd(self._desc, a["q"], a["k"], a["v"], a["g"], a["beta"], a["h0"], a["dO"], a["dhT"],
                                a["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["dbeta"], o["dh0"], sl["ws"],
                                workspace_is_fresh_from_fwd=0, stream=self._s_c)
                sl["ev_c"].record(self._s_c)
            with torch.cuda.stream(self._s_out):
                self._s_out.wait_event(sl["ev_c"])
                for k, v in self.outputs.items():
                    if v is not None:
                        self._host_slice(v, k, i).copy_(sl["out"][k], non_blocking=True)
        for s in (self._s_in, self._s_c, self._s_out):
            cur.wait_stream(s)

    def check(self) -> None:
        """Synchronise and raise if any piece recorded a device-side error."""
        torch.cuda.synchronize(self.dev)
        for sl in self._slots:
            st = binding.gdn_last_device_status(sl["ws"])
            if st != binding.GDN_OK:
                raise binding.GdnError(st, "device status")


# ---- entry points with per-channel gates ----
def to_device_channelwise(wl: Workload, device="cuda:0", want_o: bool = False) -> DeviceBuffers:
    io = _io_dtype(wl)
    dev = torch.device(device)
    t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
    inputs = dict(q=t(wl.q, io), k=t(wl.k, io), v=t(wl.v, io), dO=t(wl.dO, io), g=t(wl.gv, torch.float32),
                  b=t(wl.bv, torch.float32), w=t(wl.wv, torch.float32), h0=t(wl.h0, torch.float32),
                  dhT=t(wl.dhT, torch.float32), cu_seqlens=t(wl.cu_seqlens, torch.int32) if wl.varlen else None)
    Tt, H, N = wl.T_total, wl.H, wl.N
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
    outputs = dict(dq=z((Tt, H, wl.d_k), io), dk=z((Tt, H, wl.d_k), io), dv=z((Tt, H, wl.d_v), io),
                   dg=z((Tt, H, wl.d_k), torch.float32), db=z((Tt, H, wl.d_k), torch.float32),
                   dw=z((Tt, H, wl.d_v), torch.float32), dh0=z((N, H, wl.d_k, wl.d_v), torch.float32),
                   o=z((Tt, H, wl.d_v), io) if want_o else None,
                   hT=z((N, H, wl.d_k, wl.d_v), torch.float32) if want_o else None)
    desc = desc_for(wl)
    _, bwd_bytes = binding.gdn_workspace_bytes_channelwise(desc)
    ws = torch.empty(bwd_bytes, dtype=torch.uint8, device=dev)
    return DeviceBuffers(desc=desc, inputs=inputs, outputs=outputs, workspace=ws)


def run_fwd_channelwise(buf: DeviceBuffers, stream=None) -> None:
    i, o = buf.inputs, buf.outputs
    binding.gdn_fwd_recompute_channelwise(buf.desc, i["q"], i["k"], i["v"], i["g"], i["b"], i["w"], i["h0"],
                                          i["cu_seqlens"], o["o"], o["hT"], buf.workspace, stream=stream)


def run_bwd_channelwise(buf: DeviceBuffers, fresh: int = 0, stream=None) -> None:
    i, o = buf.inputs, buf.outputs
    binding.gdn_bwd_channelwise(buf.desc, i["q"], i["k"], i["v"], i["g"], i["b"], i["w"], i["h0"], i["dO"], i["dhT"],
                                i["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["db"], o["dw"], o["dh0"],
                                buf.workspace, workspace_is_fresh_from_fwd=fresh, stream=stream)


def backward_channelwise(wl: Workload, device="cuda:0") -> Dict[str, np.ndarray]:
    buf = to_device_channelwise(wl, device)
    run_bwd_channelwise(buf)
    return fetch(buf)
