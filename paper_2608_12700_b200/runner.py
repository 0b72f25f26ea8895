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
