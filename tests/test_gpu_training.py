"""It trains (paper Section 4.5): a tiny one-layer model whose sequence mixer is the library's recurrence is
fitted to a teacher of the same architecture.  The forward output comes from gdn_fwd_recompute, the gradients of
q, k, v and the gates from gdn_bwd on the workspace the forward left (the save-forward arm); only the projections
around the recurrence are differentiated by the framework.  Every family member of Table 2 runs as a gate setting:
LA, SSD and scalar-gate GDN through gdn_bwd, GLA, KDA and the full per-channel GDN through gdn_bwd_channelwise.
The loss must fall and stay finite."""
import pytest
import torch
import torch.nn.functional as F

from paper_2608_12700_b200 import binding

pytestmark = pytest.mark.gpu


class ScalarGateMixer(torch.autograd.Function):
    """o = recurrence(q, k, v, g, beta); tensors [B, T, H, d] / [B, T, H], contiguous, on the GPU."""

    @staticmethod
    def forward(ctx, q, k, v, g, beta, delta_rule):
        B, T, H, dk = q.shape
        dv = v.shape[-1]
        desc = binding.make_desc(B=B, T=T, H=H, d_k=dk, d_v=dv, N=B, dtype="bf16" if q.dtype == torch.bfloat16 else "f32",
                                 delta_rule=delta_rule)
        _, nbytes = binding.gdn_workspace_bytes(desc)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
        o = torch.empty_like(v)
        binding.gdn_fwd_recompute(desc, q, k, v, g, beta if delta_rule else None, None, None, o, None, ws)
        ctx.save_for_backward(q, k, v, g, beta)
        ctx.desc, ctx.ws, ctx.delta_rule = desc, ws, delta_rule
        return o

    @staticmethod
    def backward(ctx, dO):
        q, k, v, g, beta = ctx.saved_tensors
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        dg, dbeta = torch.empty_like(g), torch.zeros_like(beta)
        dr = ctx.delta_rule
        binding.gdn_bwd(ctx.desc, q, k, v, g, beta if dr else None, None, dO.contiguous(), None, None, dq, dk, dv, dg,
                        dbeta if dr else None, None, ctx.ws, workspace_is_fresh_from_fwd=1)
        assert binding.gdn_last_device_status(ctx.ws) == binding.GDN_OK
        return dq, dk, dv, dg, dbeta, None


class ChannelGateMixer(torch.autograd.Function):
    """The same with gate vectors g, b [B, T, H, d_k] and w [B, T, H, d_v]."""

    @staticmethod
    def forward(ctx, q, k, v, g, b, w):
        B, T, H, dk = q.shape
        dv = v.shape[-1]
        desc = binding.make_desc(B=B, T=T, H=H, d_k=dk, d_v=dv, N=B, dtype="bf16" if q.dtype == torch.bfloat16 else "f32")
        _, nbytes = binding.gdn_workspace_bytes_channelwise(desc)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
        o = torch.empty_like(v)
        binding.gdn_fwd_recompute_channelwise(desc, q, k, v, g, b, w, None, None, o, None, ws)
        ctx.save_for_backward(q, k, v, g, b, w)
        ctx.desc, ctx.ws = desc, ws
        return o

    @staticmethod
    def backward(ctx, dO):
        q, k, v, g, b, w = ctx.saved_tensors
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        dg, db, dw = torch.empty_like(g), torch.empty_like(b), torch.empty_like(w)
        binding.gdn_bwd_channelwise(ctx.desc, q, k, v, g, b, w, None, dO.contiguous(), None, None, dq, dk, dv, dg, db, dw,
                                    None, ctx.ws, workspace_is_fresh_from_fwd=1)
        assert binding.gdn_last_device_status(ctx.ws) == binding.GDN_OK
        return dq, dk, dv, dg, db, dw


class TinyLayer(torch.nn.Module):
    """x -> projections -> recurrence -> o.  `member` picks the gate setting (Table 2)."""

    def __init__(self, member, d_in, H, dk, dv, io, gen):
        super().__init__()
        self.member, self.H, self.dk, self.dv, self.io = member, H, dk, dv, io
        channel = member in ("gla", "kda", "gdn")
        n_g = H * dk if member in ("gla", "kda", "gdn") else H
        n_b = H * dk if member == "gdn" else H
        n_w = H * dv if member == "gdn" else H
        mk = lambda n: torch.nn.Parameter(torch.randn(d_in, n, generator=gen, device="cuda") / d_in ** 0.5)
        self.wq, self.wk, self.wv = mk(H * dk), mk(H * dk), mk(H * dv)
        self.wg, self.wb, self.ww = mk(n_g), mk(n_b), mk(n_w)
        self.channel = channel

    def forward(self, x):
        B, T, _ = x.shape
        H, dk, dv = self.H, self.dk, self.dv
        q = F.normalize((x @ self.wq).view(B, T, H, dk), dim=-1).to(self.io).contiguous()
        k = F.normalize((x @ self.wk).view(B, T, H, dk), dim=-1).to(self.io).contiguous()
        v = (x @ self.wv).view(B, T, H, dv).to(self.io).contiguous()
        m = self.member
        if not self.channel:
            g = -0.1 * F.softplus(x @ self.wg).view(B, T, H)
            if m == "la":
                g = torch.zeros_like(g)                       # no decay, no delta rule
            beta = torch.sigmoid(x @ self.wb).view(B, T, H)
            o = ScalarGateMixer.apply(q, k, v, g.contiguous(), beta.contiguous(), 1 if m == "gdn_scalar" else 0)
        else:
            g = (-0.1 * F.softplus(x @ self.wg)).view(B, T, H, dk).contiguous()
            if m == "gla":
                b = torch.zeros(B, T, H, dk, device=x.device)
                w = torch.ones(B, T, H, dv, device=x.device)
            elif m == "kda":
                beta = torch.sigmoid(x @ self.wb).view(B, T, H, 1)
                b, w = beta.expand(B, T, H, dk).contiguous(), beta.expand(B, T, H, dv).contiguous()
            else:
                b = torch.sigmoid(x @ self.wb).view(B, T, H, dk).contiguous()
                w = torch.sigmoid(x @ self.ww).view(B, T, H, dv).contiguous()
            o = ChannelGateMixer.apply(q, k, v, g, b, w)
        return o.float()


def fit(member, io=torch.float32, d=64, steps=60):
    gen = torch.Generator(device="cuda").manual_seed(1234)
    B, T, H, d_in = 2, 128, 2, 32
    x = torch.randn(B, T, d_in, generator=gen, device="cuda")
    teacher = TinyLayer(member, d_in, H, d, d, io, gen)
    student = TinyLayer(member, d_in, H, d, d, io, gen)
    with torch.no_grad():
        target = teacher(x)
    opt = torch.optim.Adam(student.parameters(), lr=1e-2)
    losses = []
    for _ in range(steps):
        opt.zero_grad()
        loss = F.mse_loss(student(x), target)
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    return losses


@pytest.mark.parametrize("member", ["la", "ssd", "gdn_scalar", "gla", "kda", "gdn"])
def test_every_family_member_trains_fp32(member):
    losses = fit(member)
    print(member, [round(l, 5) for l in losses[::10]], round(losses[-1], 5))
    assert all(l == l and l < float("inf") for l in losses)
    assert losses[-1] < 0.6 * losses[0], losses


def test_gdn_trains_through_the_tensor_core_kernels():
    """bf16 I/O, d_k = d_v = 128: forward and backward run on the tcgen05 family."""
    assert binding.gdn_kernel_path(binding.make_desc(B=2, T=128, H=2, d_k=128, d_v=128, N=2, dtype="bf16")) == "tcgen05_bf16"
    losses = fit("gdn_scalar", io=torch.bfloat16, d=128)
    print("gdn bf16", [round(l, 5) for l in losses[::10]], round(losses[-1], 5))
    assert all(l == l and l < float("inf") for l in losses)
    assert losses[-1] < 0.6 * losses[0], losses
