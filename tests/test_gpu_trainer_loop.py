"""The library inside a training loop: W data-parallel replicas of a small least-squares model,
gradients from PyTorch autograd written into the [W][N] table, one `la_step_grads` per optimizer
step.  Checked against a plain PyTorch (fp32) restatement of Algorithm 3 and against the paper's
qualitative claim that the loss goes down with H > 1."""
import numpy as np
import pytest

from paper_1911_09030_b200 import local_adaalter as la

pytestmark = pytest.mark.gpu


def test_autograd_training_loop_matches_plain_pytorch():
    import torch
    torch.manual_seed(0)
    W, d_in, d_out, batch, H, T = 4, 32, 8, 64, 4, 60
    N = d_in * d_out + d_out
    eta, eps, b0sq = 0.5, 1.0, 1.0
    true_w = torch.randn(d_in, d_out, device="cuda")

    def batch_for(worker, step):
        g = torch.Generator(device="cuda").manual_seed(1000 * worker + step)
        x = torch.randn(batch, d_in, device="cuda", generator=g)
        y = x @ true_w + 0.01 * torch.randn(batch, d_out, device="cuda", generator=g)
        return x, y

    def loss_fn(flat, x, y):
        w = flat[: d_in * d_out].view(d_in, d_out)
        b = flat[d_in * d_out:]
        return ((x @ w + b - y) ** 2).mean()

    ctx = la.LocalAdaAlter([d_in * d_out, d_out], W, eta, eps, H, b0sq=b0sq)
    ctx.set_init(None, b0sq)
    ctx.set_fusion(la.LA_FUSE_STEP_SYNC)
    # plain PyTorch restatement of Algorithm 3
    X = torch.zeros(W, N, device="cuda")
    B2 = torch.full((W, N), b0sq, device="cuda")
    Bs = torch.full((N,), b0sq, device="cuda")
    tp = 0
    losses = []
    params = torch.zeros(W, N, device="cuda")          # what the "model" sees each step
    for step in range(1, T + 1):
        grads = torch.empty(W, N, device="cuda")
        step_loss = 0.0
        for i in range(W):
            p = params[i].clone().requires_grad_(True)
            x, y = batch_for(i, step)
            l = loss_fn(p, x, y)
            l.backward()
            grads[i] = p.grad
            step_loss += float(l.detach())
        losses.append(step_loss / W)
        # library
        ctx.step_grads(grads.data_ptr(), la.LA_F32)
        # reference
        tp += 1
        r = eta / torch.sqrt(Bs + tp * eps * eps)
        X = X - r * grads
        B2 = B2 + grads * grads
        if tp == H:
            X = X.mean(0, keepdim=True).expand(W, N).clone()
            B2 = B2.mean(0, keepdim=True).expand(W, N).clone()
            Bs = B2[0].clone()
            tp = 0
        ctx.sync_stream()
        for i in range(W):
            params[i] = torch.from_numpy(ctx.read_state(i)[0]).cuda()
        torch.testing.assert_close(params, X, rtol=2e-4, atol=2e-5)
    assert ctx.get_counters() == (T, T % H, T // H)
    assert losses[-1] < 0.05 * losses[0]               # it trains
    off, sz = ctx.tensor_range(1)
    assert (off, sz) == (d_in * d_out, d_out)
