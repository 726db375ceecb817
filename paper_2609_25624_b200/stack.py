"""Synthetic decode-step linear stack of a Llama-3-8B-architecture model (harness, not a model).

32 layers x (qkv 4096->6144, o 4096->4096, gate_up 4096->28672, down 14336->4096) + LM head
4096->128256, about 15 GB of BF16 weights.  Only the linear layers are the library's kernels; the
glue between them is elementwise (slice, multiply by a constant -- a test-only kernel that keeps the
programmatic-dependent-launch chain intact -- and a gather), chosen so that nothing
order-dependent is introduced and the activations stay near N(0, 1):

    q  = c1 * qkv(x)[:, :4096]        c1 = c2 = c3 = 1 / (0.02 * sqrt(4096))
    o  = c2 * o_proj(q)               c4 = 1 / (0.02 * sqrt(14336))
    h  = c3 * gate_up(o)[:, :14336]
    x' = c4 * down(h)
    logits = lm_head(x_after_32_layers);  next x row = 50 * up(W_lm[argmax(logits)])

so the 64 steps form a real autoregressive chain in which one flipped bit would propagate.
"""
import hashlib
import math

import numpy as np
import torch

from . import binding as B
from . import inputs

HIDDEN, QKV, FFN, VOCAB = 4096, 6144, 14336, 128256
C_IN = np.float32(1.0 / (0.02 * math.sqrt(4096.0)))
C_DOWN = np.float32(1.0 / (0.02 * math.sqrt(14336.0)))
EMBED_SCALE = np.float32(50.0)
SHAPES = {"qkv": (HIDDEN, QKV), "o": (HIDDEN, HIDDEN), "gate_up": (HIDDEN, 2 * FFN), "down": (FFN, HIDDEN),
          "lm_head": (HIDDEN, VOCAB)}          # name -> (K, N)


def weight_seed(layer, name):
    return inputs.named_seed(f"L{layer}.{name}")


class LinearStack:
    """Holds the device weights and one set of plans per batch size."""

    def __init__(self, n_layers=32, device="cuda"):
        self.n_layers = n_layers
        self.device = device
        self.weights = [dict() for _ in range(n_layers)]
        self.lm_head = None
        self._plans = {}

    def load_cpu_seeded(self, on_matrix=None):
        """Seeded CPU generation (the paper's probe methodology), matrix by matrix.  `on_matrix(layer,
        name, W_cpu)` lets a test look at each CPU matrix before it is dropped."""
        for layer in range(self.n_layers):
            for name in ("qkv", "o", "gate_up", "down"):
                K, N = SHAPES[name]
                W = inputs.make_weight(N, K, weight_seed(layer, name))
                self.weights[layer][name] = W.to(self.device)
                if on_matrix:
                    on_matrix(layer, name, W)
        K, N = SHAPES["lm_head"]
        W = inputs.make_weight(N, K, inputs.named_seed("lm_head"))
        self.lm_head = W.to(self.device)
        if on_matrix:
            on_matrix(-1, "lm_head", W)

    def load_device_random(self, seed=0):
        """Weights drawn on the device (for timing only: same distribution, not the seeded CPU bits)."""
        g = torch.Generator(device=self.device).manual_seed(seed)
        for layer in range(self.n_layers):
            for name in ("qkv", "o", "gate_up", "down"):
                K, N = SHAPES[name]
                self.weights[layer][name] = (0.02 * torch.randn(N, K, device=self.device, generator=g)).to(torch.bfloat16)
        K, N = SHAPES["lm_head"]
        self.lm_head = (0.02 * torch.randn(N, K, device=self.device, generator=g)).to(torch.bfloat16)

    def plans(self, M, key=0):
        k = (M, key)
        if k not in self._plans:
            self._plans[k] = {name: B.det_linear_plan(M, N, K) for name, (K, N) in SHAPES.items()}
        return self._plans[k]

    def close(self):
        for ps in self._plans.values():
            for p in ps.values():
                p.close()
        self._plans = {}

    def linear(self, plans, name, W, x, stream=None):
        K, N = SHAPES[name]
        y = torch.empty(x.shape[0], N, dtype=torch.float32, device=x.device)
        B.det_linear_run(plans[name], x, W, None, y, stream=stream)
        return y

    def layer(self, plans, layer, x, stream=None, trace=None):
        w = self.weights[layer]
        y = self.linear(plans, "qkv", w["qkv"], x, stream)
        if trace is not None:
            trace(layer, "qkv", x, y)
        q = B.det_test_scale_cols(y, HIDDEN, float(C_IN), stream)
        y = self.linear(plans, "o", w["o"], q, stream)
        if trace is not None:
            trace(layer, "o", q, y)
        o = B.det_test_scale_cols(y, HIDDEN, float(C_IN), stream)
        y = self.linear(plans, "gate_up", w["gate_up"], o, stream)
        if trace is not None:
            trace(layer, "gate_up", o, y)
        h = B.det_test_scale_cols(y, FFN, float(C_IN), stream)
        y = self.linear(plans, "down", w["down"], h, stream)
        if trace is not None:
            trace(layer, "down", h, y)
        return B.det_test_scale_cols(y, HIDDEN, float(C_DOWN), stream)

    def step(self, plans, x, stream=None, trace=None):
        """One decode step: x [M, 4096] -> (logits [M, 128256], argmax [M] int32, next x)."""
        for layer in range(self.n_layers):
            x = self.layer(plans, layer, x, stream, trace)
        logits = self.linear(plans, "lm_head", self.lm_head, x, stream)
        if trace is not None:
            trace(-1, "lm_head", x, logits)
        idx = torch.empty(x.shape[0], dtype=torch.int32, device=x.device)
        B.det_argmax_rows(logits, idx, stream=stream)
        nxt = self.lm_head[idx.long()].to(torch.float32) * float(EMBED_SCALE)
        return logits, idx, nxt

    def run(self, x0, steps, key=0, stream=None):
        """Run `steps` decode steps from x0; returns (list of SHA-256 digests of each step's logits,
        list of argmax lists)."""
        M = x0.shape[0]
        plans = self.plans(M, key)
        x = x0.clone()
        digests, tokens = [], []
        for _ in range(steps):
            logits, idx, x = self.step(plans, x, stream)
            digests.append(hashlib.sha256(logits.cpu().numpy().tobytes()).hexdigest())
            tokens.append(idx.cpu().tolist())
        for p in plans.values():
            B.det_linear_plan_check(p, stream=stream)
        return digests, tokens


def initial_activations(M, seed=1234):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(M, HIDDEN, generator=g)
