"""Host-side helpers of the benchmark: clock sampling, roofline bookkeeping, cross-rank aggregation.

Nothing here touches the method's arithmetic.  The roofline bookkeeping counts what the *method* has to
move and multiply (inputs read once, gradients written once, one pass over the products of the chunked
formulation); workspace traffic is overhead and deliberately not counted.
"""
from __future__ import annotations

import json
import os
import threading
import time
from typing import Dict, List, Optional

C = 64  # chunk length


# ---------------------------------------------------------------------------------------------------
# peaks
# ---------------------------------------------------------------------------------------------------
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks(repo_root: str) -> Dict:
    """Measured peaks of this machine's B200 (generated file), else the stated fallback."""
    path = os.path.join(repo_root, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(FALLBACK_PEAKS, source="fallback")


# ---------------------------------------------------------------------------------------------------
# algorithmic work
# ---------------------------------------------------------------------------------------------------
def path_alg_bytes(*, token_heads: int, chains: int, d_k: int, d_v: int, io_bytes: int, delta_rule: int,
                   has_h0: bool, has_dhT: bool, writes_dh0: bool = True) -> int:
    """Bytes the method must move: q,k,v,dO,g(,beta) read once; dq,dk,dv,dg(,dbeta) written once; states once."""
    gates = 2 if delta_rule else 1
    per_th = (2 * d_k + 2 * d_v) * io_bytes + 4 * gates + (2 * d_k + d_v) * io_bytes + 4 * gates
    states = (int(has_h0) + int(has_dhT) + int(writes_dh0)) * d_k * d_v * 4
    return token_heads * per_th + chains * states


def path_alg_flops(*, chunk_heads: int, d_k: int, d_v: int, delta_rule: int) -> float:
    """Flops of one pass over the chunked formulation, a product with a triangular operand or a
    triangular result counted at half (2*m*n*k/2)."""
    tri_k, tri_v, dense = C * C * d_k, C * C * d_v, 2 * C * d_k * d_v
    if delta_rule:
        # triangular, contraction over d_k or a [C, d_k] result: K K^T, W, Q K^T, (dP.D)K, (dP.D)^T Q, T^T dW,
        #   dXk W^T, (bG)K, (bG)^T K ; over d_v or a [C, d_v] result: U~, P^T dO, dO U^T, T^T dU, dXv U~^T
        # dense: W h, Kb^T U, Kb dh, Q~^T dO, W^T dU, (Gam dO) h^T, U dh^T, dU h^T ; inverse ~ 2 C^3 / 3
        return chunk_heads * (9 * tri_k + 5 * tri_v + 8 * dense + 2 * C ** 3 / 3)
    # delta rule off: Q K^T, (dP.D)K, (dP.D)^T Q | P^T dO, dO V^T | Kb^T V, Kb dh, Q~^T dO, (Gam dO) h^T, V dh^T
    return chunk_heads * (3 * tri_k + 2 * tri_v + 5 * dense)


def roofline_times(alg_bytes: float, alg_flops: float, peaks: Dict, sustained: bool = False):
    t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = alg_flops / ((peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]) * 1e12)
    return t_hbm, t_tc


# ---------------------------------------------------------------------------------------------------
# clocks (NVML, read-only)
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU while a timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.samples: List[int] = []
        self.reason_bits = 0
        self.max_mhz: Optional[int] = None
        self.power_w: List[float] = []
        self._stop = threading.Event()
        self._thr: Optional[threading.Thread] = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _one(self):
        nv = self._nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            self.power_w.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._one()
            time.sleep(self.period)

    def start(self):
        if self._h is None:
            return
        self._stop.clear()
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def stop(self):
        if self._h is None:
            return
        self._one()
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self) -> Dict:
        if self._h is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        s = sorted(self.samples)
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(s),
                "power_w_max": round(max(self.power_w), 1) if self.power_w else None}


# ---------------------------------------------------------------------------------------------------
# cross-rank aggregation (one process per GPU, independent batches, no data-path collective)
# ---------------------------------------------------------------------------------------------------
def aggregate_over_ranks(elapsed_ms: float, units: float, dist=None, device=None):
    """Returns (max elapsed over ranks, total units over ranks).  `dist` is torch.distributed or None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
