"""Seeded synthetic inputs for the gated-delta-rule (GDN) backward.

This module only draws random numbers and rounds them to the I/O dtype.  It holds
none of the method's arithmetic, so both the CUDA path and the CPU oracle may be
fed from it without sharing any computation.

All tensors are returned as float32 numpy arrays whose *values* are exactly
representable in the workload's I/O dtype (bf16 inputs are rounded once, to
nearest even, before anybody sees them).  Layout is token-major and packed:

    q, k        [T_total, H, d_k]
    v, dO       [T_total, H, d_v]
    g, beta     [T_total, H]          (float32 in every configuration)
    h0, dhT     [N, H, d_k, d_v]      (float32, or None)
    cu_seqlens  int32 [N + 1]

A fixed-length batch of B sequences of T tokens is the packed case with
cu_seqlens = [0, T, 2T, ...], which is byte-identical to a [B, T, H, d] tensor.

Value distributions (the five benchmark configurations): q, k ~ N(0,1) then
L2-normalised over the feature axis per (token, head); v, dO ~ N(0,1);
beta = sigmoid(N(0,1)); g = -g_scale * softplus(N(0,1)); h0, dhT ~ N(0, 0.1^2).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even), keep float32 storage."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    # NaN/Inf: keep the top 16 bits (a NaN stays a NaN)
    special = (u & np.uint32(0x7F800000)) == np.uint32(0x7F800000)
    r = np.where(special, u & np.uint32(0xFFFF0000) | np.where((u & np.uint32(0x007FFFFF)) != 0, np.uint32(0x00400000), np.uint32(0)), r)
    return r.astype(np.uint32).view(np.float32).reshape(x.shape)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit pattern of already-bf16-representable float32 values."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    name: str
    dtype: str                 # "f32" | "bf16": dtype of q, k, v, dO and of dq, dk, dv
    B: int                     # batch dimension of the [B, T, H, d] view (1 when packed)
    T: int                     # tokens per batch row of that view
    H: int
    d_k: int
    d_v: int
    chunk: int
    scale: float
    delta_rule: int            # 1: erase = write = beta;  0: erase = 0, write = 1 (beta unused)
    seed: int
    cu_seqlens: np.ndarray     # int32 [N + 1]
    varlen: bool               # True when cu_seqlens must be passed explicitly
    q: np.ndarray = field(repr=False, default=None)
    k: np.ndarray = field(repr=False, default=None)
    v: np.ndarray = field(repr=False, default=None)
    dO: np.ndarray = field(repr=False, default=None)
    g: np.ndarray = field(repr=False, default=None)
    beta: Optional[np.ndarray] = field(repr=False, default=None)
    h0: Optional[np.ndarray] = field(repr=False, default=None)
    dhT: Optional[np.ndarray] = field(repr=False, default=None)
    # channel-wise workloads only: gate vectors g, b [T_total, H, d_k] and w [T_total, H, d_v] (float32)
    gv: Optional[np.ndarray] = field(repr=False, default=None)
    bv: Optional[np.ndarray] = field(repr=False, default=None)
    wv: Optional[np.ndarray] = field(repr=False, default=None)

    @property
    def N(self) -> int:
        return len(self.cu_seqlens) - 1

    @property
    def T_total(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def tokens(self) -> int:
        """Tokens counted by the throughput metric (heads are not multiplied in)."""
        return self.T_total

    def seq_lengths(self) -> np.ndarray:
        return np.diff(self.cu_seqlens)

    def n_chunks(self) -> int:
        return int(np.sum((self.seq_lengths() + self.chunk - 1) // self.chunk))

    def take_heads(self, heads) -> "Workload":
        """A smaller workload holding only the listed heads (chains are independent per head)."""
        heads = list(heads)
        sl = lambda a: None if a is None else np.ascontiguousarray(a[:, heads])
        return Workload(
            name=self.name + f"[heads={heads}]", dtype=self.dtype, B=self.B, T=self.T, H=len(heads),
            d_k=self.d_k, d_v=self.d_v, chunk=self.chunk, scale=self.scale, delta_rule=self.delta_rule,
            seed=self.seed, cu_seqlens=self.cu_seqlens, varlen=self.varlen,
            q=sl(self.q), k=sl(self.k), v=sl(self.v), dO=sl(self.dO), g=sl(self.g), beta=sl(self.beta),
            h0=sl(self.h0), dhT=sl(self.dhT), gv=sl(self.gv), bv=sl(self.bv), wv=sl(self.wv))


def _softplus(z):
    return np.logaddexp(0.0, z)


def make_workload(name: str, *, dtype: str, H: int, d_k: int, d_v: int, seed: int,
                  B: int = 1, T: int = 0, lengths=None, g_scale: float = 0.1,
                  delta_rule: int = 1, states: bool = False, state_std: float = 0.1,
                  scale: float = 1.0, chunk: int = 64) -> Workload:
    """Draw one workload.  Either (B, T) for a fixed-length batch or `lengths` for a packed one."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if lengths is None:
        cu = np.arange(B + 1, dtype=np.int64) * T
        varlen = False
    else:
        lengths = np.asarray(lengths, dtype=np.int64)
        cu = np.concatenate([[0], np.cumsum(lengths)])
        B, T, varlen = 1, int(cu[-1]), True
    Tt, N = int(cu[-1]), len(cu) - 1

    def normal(shape):
        return rng.standard_normal(shape, dtype=np.float32)

    def unit(shape):
        x = normal(shape)
        nrm = np.sqrt(np.sum(x.astype(np.float64) ** 2, axis=-1, keepdims=True))
        return (x / np.maximum(nrm, 1e-30)).astype(np.float32)

    q = unit((Tt, H, d_k))
    k = unit((Tt, H, d_k))
    v = normal((Tt, H, d_v))
    dO = normal((Tt, H, d_v))
    beta = (1.0 / (1.0 + np.exp(-normal((Tt, H)).astype(np.float64)))).astype(np.float32)
    g = (-g_scale * _softplus(normal((Tt, H)).astype(np.float64))).astype(np.float32)
    h0 = dhT = None
    if states:
        h0 = (state_std * normal((N, H, d_k, d_v))).astype(np.float32)
        dhT = (state_std * normal((N, H, d_k, d_v))).astype(np.float32)
    if dtype == "bf16":
        q, k, v, dO = (round_to_bf16(a) for a in (q, k, v, dO))
    elif dtype != "f32":
        raise ValueError(f"unknown dtype {dtype!r}")
    return Workload(name=name, dtype=dtype, B=B, T=T, H=H, d_k=d_k, d_v=d_v, chunk=chunk, scale=scale,
                    delta_rule=delta_rule, seed=seed, cu_seqlens=cu.astype(np.int32), varlen=varlen,
                    q=q, k=k, v=v, dO=dO, g=g, beta=beta if delta_rule else None, h0=h0, dhT=dhT)


def make_channelwise(name: str, *, member: str = "gdn", gate_seed: int = 0, **kw) -> Workload:
    """A workload for the entry points with per-channel gates: the tensors of make_workload plus gate vectors
    gv, bv [T_total, H, d_k] and wv [T_total, H, d_v], drawn like their scalar counterparts (log-decay
    -g_scale * softplus(N(0,1)) per channel, erase and write gates sigmoid(N(0,1))).  `member` picks the row of the
    family table: "gdn" independent vectors, "kda" one beta per token broadcast to both gates, "gla" erase 0, write 1."""
    g_scale = kw.get("g_scale", 0.1)
    wl = make_workload(name, **kw)
    rng = np.random.Generator(np.random.PCG64([wl.seed, 7919 + gate_seed]))
    Tt, H = wl.T_total, wl.H
    sig = lambda z: (1.0 / (1.0 + np.exp(-z.astype(np.float64)))).astype(np.float32)
    wl.gv = (-g_scale * _softplus(rng.standard_normal((Tt, H, wl.d_k), dtype=np.float32).astype(np.float64))).astype(np.float32)
    if member == "gdn":
        wl.bv = sig(rng.standard_normal((Tt, H, wl.d_k), dtype=np.float32))
        wl.wv = sig(rng.standard_normal((Tt, H, wl.d_v), dtype=np.float32))
    elif member == "kda":
        beta = sig(rng.standard_normal((Tt, H, 1), dtype=np.float32))
        wl.bv = np.ascontiguousarray(np.broadcast_to(beta, (Tt, H, wl.d_k)))
        wl.wv = np.ascontiguousarray(np.broadcast_to(beta, (Tt, H, wl.d_v)))
    elif member == "gla":
        wl.bv = np.zeros((Tt, H, wl.d_k), dtype=np.float32)
        wl.wv = np.ones((Tt, H, wl.d_v), dtype=np.float32)
    else:
        raise ValueError(f"unknown family member {member!r}")
    wl.g = None
    wl.beta = None
    return wl


def draw_packed_lengths(seed: int, n_seq: int = 8, lo: int = 256, hi: int = 8192, total: int = 32768):
    """n_seq lengths, each uniform in [lo, hi], conditioned on summing to `total`.

    Rejection sampling: draw n_seq - 1 lengths uniformly, set the last to the remainder, accept when
    the remainder also lies in [lo, hi].  The lengths are in general not multiples of the chunk.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    while True:
        first = rng.integers(lo, hi + 1, size=n_seq - 1)
        last = total - int(first.sum())
        if lo <= last <= hi:
            return [int(x) for x in first] + [last]


CONFIG_NAMES = ["cfg0_f32_small", "cfg1_bf16_train", "cfg2_bf16_scalar_gate", "cfg3_bf16_long", "cfg4_bf16_varlen"]


def config(i: int, *, heads: Optional[int] = None) -> Workload:
    """The five benchmark configurations (index 0..4).  `heads` overrides H (used to bound CPU work)."""
    if i == 0:
        return make_workload(CONFIG_NAMES[0], dtype="f32", B=1, T=128, H=heads or 2, d_k=64, d_v=64, seed=0)
    if i == 1:
        return make_workload(CONFIG_NAMES[1], dtype="bf16", B=4, T=2048, H=heads or 16, d_k=128, d_v=128,
                             seed=1, states=True)
    if i == 2:
        return make_workload(CONFIG_NAMES[2], dtype="bf16", B=8, T=4096, H=heads or 32, d_k=64, d_v=64,
                             seed=2, g_scale=0.05, delta_rule=0)
    if i == 3:
        return make_workload(CONFIG_NAMES[3], dtype="bf16", B=1, T=16384, H=heads or 16, d_k=128, d_v=128,
                             seed=3, states=True)
    if i == 4:
        return make_workload(CONFIG_NAMES[4], dtype="bf16", H=heads or 32, d_k=128, d_v=128, seed=4,
                             lengths=draw_packed_lengths(4), states=True)
    raise ValueError("config index must be 0..4")


def device_inputs(*, B: int, T: int, H: int, d_k: int, d_v: int, dtype: str, seed: int, device="cuda:0",
                  g_scale: float = 0.1, delta_rule: int = 1, states: bool = False, state_std: float = 0.1):
    """The same value distributions as `make_workload`, drawn on the device with torch's generator, one batch row at a
    time: for inputs too large to be drawn on the host and uploaded (tensors beyond 4 GiB).  Returns a dict of torch
    tensors q, k [B*T, H, d_k], v, dO [B*T, H, d_v] (I/O dtype), g, beta [B*T, H] (fp32; beta None without the delta
    rule), h0, dhT [B, H, d_k, d_v] (fp32, or None).  Whoever wants a CPU result copies the rows it needs to the host."""
    import torch

    dev = torch.device(device)
    io = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    q = torch.empty((B * T, H, d_k), dtype=io, device=dev)
    k = torch.empty_like(q)
    v = torch.empty((B * T, H, d_v), dtype=io, device=dev)
    dO = torch.empty_like(v)
    g = torch.empty((B * T, H), dtype=torch.float32, device=dev)
    beta = torch.empty_like(g) if delta_rule else None
    normal = lambda *shape: torch.randn(shape, generator=gen, device=dev, dtype=torch.float32)
    for n in range(B):
        rows = slice(n * T, (n + 1) * T)
        for dst, d in ((q, d_k), (k, d_k)):
            x = normal(T, H, d)
            dst[rows] = (x / x.norm(dim=-1, keepdim=True).clamp_min(1e-30)).to(io)
        v[rows] = normal(T, H, d_v).to(io)
        dO[rows] = normal(T, H, d_v).to(io)
        g[rows] = -g_scale * torch.nn.functional.softplus(normal(T, H))
        if delta_rule:
            beta[rows] = torch.sigmoid(normal(T, H))
    h0 = dhT = None
    if states:
        h0 = state_std * normal(B, H, d_k, d_v)
        dhT = state_std * normal(B, H, d_k, d_v)
    return dict(q=q, k=k, v=v, dO=dO, g=g, beta=beta, h0=h0, dhT=dhT)
