"""One DeiT-Small transformer block (pre-LayerNorm: attention + MLP, D = 384, 12 heads, MLP 1536) run around the
MXFP4 linear layer: the harness of the fifth workload.

Everything that is not a linear layer (LayerNorm, softmax attention, GELU, residual additions) is plain PyTorch in bf16
with autograd; the four linear layers (qkv, proj, fc1, fc2) go through the library's forward and backward entry points,
with the Q-EMA weight quantizer and the per-element oscillation counters run once per step.  Each linear layer records
the tensors it saw (X, dY) and produced (Y, dX, dW), so that a test can replay them through the CPU oracle.

This module holds no arithmetic of the method: it only decides which tensors go into which library call.
"""
import numpy as np
import torch

import workloads

D_MODEL, HEADS, D_MLP, TOKENS = 384, 12, 1536, 197
CONFIG = 5   # seeds and layer shapes of workloads.CONFIGS[5]: qkv, proj, fc1, fc2


class MxLinear:
    """A linear layer whose products and quantizers run in the library.  State: bf16 weight, FP32 EMA of it, the
    oscillation-counter buffers, the quantized weight of this step and its backward operand Q4."""

    def __init__(self, mx, name, w, seed, beta=0.998):
        self.mx, self.name, self.seed, self.beta = mx, name, seed, beta
        self.w = w                                      # bf16 [N, K], device
        self.N, self.K = w.shape
        self.ema = w.float().contiguous()
        self.wq = mx.QMat(self.N, self.K)
        self.wq_t = mx.QMat(self.K, self.N)
        self.osc = mx.OscState(w.clone(), mx.quantize(w), torch.zeros(w.shape, device=w.device), torch.zeros(w.shape, device=w.device))
        self.status = mx.new_status()
        self.record = None                              # tensors of the last step, for the replay
        self.ws = None

    def weight_step(self):
        """Once per optimizer step: Q-EMA (Algorithm 1) with its EMA update and the counters of Sec. 6.1, then Q4."""
        self.mx.qema_quantize(self.w, self.ema, beta=self.beta, update_ema=True, osc=self.osc, out=self.wq, dev_status=self.status)
        self.mx.quantize_t(self.wq, rounding=1, seed=self.seed, stream_id=4, out=self.wq_t, dev_status=self.status)

    def __call__(self, x):
        return _MxLinearFn.apply(x, self)


class _MxLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, layer):
        mx = layer.mx
        x2 = x.reshape(-1, layer.K)
        M = x2.shape[0]
        lctx = mx.LinearCtx(mx.QMat(M, layer.K), layer.wq, xq_t=mx.QMat(layer.K, M), seed=layer.seed, wq_t=layer.wq_t)
        y, _ = mx.linear_fwd(x2, wq=layer.wq, ctx=lctx, dev_status=layer.status)
        ctx.layer, ctx.lctx, ctx.shape = layer, lctx, x.shape
        layer.record = dict(x=x2.detach(), y=y, ctx=lctx)
        return y.reshape(*x.shape[:-1], layer.N)

    @staticmethod
    def backward(ctx, dy):
        layer, mx = ctx.layer, ctx.layer.mx
        dy2 = dy.reshape(-1, layer.N).contiguous()
        M = dy2.shape[0]
        if layer.ws is None or layer.ws.numel() < mx.linear_workspace_bytes(M, layer.K, layer.N):
            layer.ws = torch.empty(mx.linear_workspace_bytes(M, layer.K, layer.N), dtype=torch.uint8, device=dy.device)
        dx, dw = mx.linear_bwd(dy2, ctx.lctx, layer.seed, workspace=layer.ws, dev_status=layer.status)
        layer.record.update(dy=dy2, dx=dx, dw=dw)
        return dx.reshape(ctx.shape), None


class Block:
    """x -> x + proj(attention(qkv(LN1(x)))) -> . + fc2(GELU(fc1(LN2(.))))"""

    def __init__(self, mx, device="cuda"):
        names = ["qkv", "proj", "fc1", "fc2"]
        self.layers = {}
        for li, (name, L) in enumerate(zip(names, workloads.CONFIGS[CONFIG])):
            w = torch.from_numpy(workloads.make_w(L, workloads.tensor_seed(CONFIG, li, "W"))).to(torch.bfloat16).to(device)
            self.layers[name] = MxLinear(mx, L.name, w, workloads.sr_seed(CONFIG, li))
        self.ln1 = torch.nn.LayerNorm(D_MODEL, device=device, dtype=torch.bfloat16)   # gamma = 1, beta = 0
        self.ln2 = torch.nn.LayerNorm(D_MODEL, device=device, dtype=torch.bfloat16)

    def weight_step(self):
        for layer in self.layers.values():
            layer.weight_step()

    def perturb_weights(self, seed, std=2e-5):
        """A small seeded move of every weight (what an optimizer step would do), so that EMA and weight differ."""
        for i, layer in enumerate(self.layers.values()):
            rng = np.random.Generator(np.random.PCG64(seed + i))
            d = torch.from_numpy(rng.standard_normal(layer.w.shape, dtype=np.float32) * np.float32(std)).to(layer.w.device)
            layer.w.copy_((layer.w.float() + d).to(torch.bfloat16))

    def forward(self, x):
        B, T, D = x.shape
        L = self.layers
        qkv = L["qkv"](self.ln1(x)).reshape(B, T, 3, HEADS, D // HEADS).permute(2, 0, 3, 1, 4)
        att = torch.nn.functional.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2])
        x = x + L["proj"](att.transpose(1, 2).reshape(B, T, D))
        return x + L["fc2"](torch.nn.functional.gelu(L["fc1"](self.ln2(x))))

    def step(self, x, dout):
        """One training step of the block's linear layers: weight quantizers, forward, backward.  Returns (out, dx)."""
        self.weight_step()
        x = x.detach().requires_grad_(True)
        out = self.forward(x)
        out.backward(dout)
        return out.detach(), x.grad


def make_block_inputs(batch, device="cuda"):
    """Tokens [batch, 197, 384] ~ N(0, 1) and the upstream gradient 1e-3 * Student-t(3), seeded like the other workloads."""
    rng = np.random.Generator(np.random.PCG64(workloads.tensor_seed(CONFIG, 0, "X")))
    x = workloads.round_to_bf16(rng.standard_normal((batch, TOKENS, D_MODEL), dtype=np.float32))
    rng = np.random.Generator(np.random.PCG64(workloads.tensor_seed(CONFIG, 3, "dY")))
    z = rng.standard_normal((batch, TOKENS, D_MODEL), dtype=np.float32)
    c = sum(rng.standard_normal((batch, TOKENS, D_MODEL), dtype=np.float32) ** 2 for _ in range(3))
    dout = workloads.round_to_bf16(z / np.sqrt(c / 3.0) * np.float32(1e-3))
    to = lambda a: torch.from_numpy(a).to(torch.bfloat16).to(device)  # noqa: E731
    return to(x), to(dout)
