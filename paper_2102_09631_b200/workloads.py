"""Seeded synthetic workloads: the (A, Delta, Q0) tensors that both the CUDA library and
the CPU oracle are fed with.

This module holds none of the method's arithmetic (no power iteration, no factor
product, no byte formula): it only manufactures layer inputs ``A_s`` (N x h_in), output
errors ``D_s`` (N x h_out) and random start blocks ``Q0_s`` (r x h_out) with the shapes,
value distributions and spectral structure of the workloads the paper trains (a ReLU
MLP on 784-pixel images, transformer encoders), because none of its datasets is needed
to exercise the per-layer path: throughput of the fixed-rank path does not depend on
the values, and parity is asserted on whatever seeded tensors both sides read.

Generators:
  * ``gaussian_layer``   -- A, D ~ N(0,1), the smallest parity case.
  * ``mlp_layers``       -- a 784-1024-1024-10 ReLU MLP with softmax cross-entropy
                            (Eq. 1 and the backward recursion of Sec. 3.1), written out by
                            hand in float64; returns the (A, D) of its three linear layers.
  * ``encoder_layers``   -- one transformer encoder layer run forward/backward with
                            autograd hooks on its six linear projections.
  * ``decaying_layer``   -- N(0,1) activations and errors with a planted 1/k spectrum
                            plus a noise floor, scaled by 1/(S*N) like a mean loss; the
                            stand-in for deep transformer stacks at full size.
  * ``start_block``      -- the N(0,1) start vectors of Algorithm 2.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import torch

SEED_BASE = 0x0DAD0000


def seed_for(config: int, layer: int = 0, site: int = 0) -> int:
    return SEED_BASE + 1000 * config + 10 * layer + site


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


@dataclasses.dataclass(frozen=True)
class LayerShape:
    name: str
    h_in: int
    h_out: int
    count: int = 1  # how many linear layers of this shape the network has


@dataclasses.dataclass(frozen=True)
class Config:
    """One benchmark configuration: S sites, N rows per site and layer, rank and iterations."""
    index: int
    name: str
    S: int
    N: int
    dtype: str  # "f32" or "bf16": storage type of A and D
    r: int
    iters: int
    layers: Tuple[LayerShape, ...]
    blocks: int = 1  # repetitions of `layers` in the full network

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def n_layers(self) -> int:
        return self.blocks * sum(l.count for l in self.layers)


CONFIGS = {
    1: Config(1, "linear-64x32", S=2, N=16, dtype="f32", r=4, iters=2,
              layers=(LayerShape("linear", 64, 32),)),
    2: Config(2, "mlp-784-1024-1024-10", S=4, N=128, dtype="f32", r=8, iters=3,
              layers=(LayerShape("fc1", 784, 1024), LayerShape("fc2", 1024, 1024), LayerShape("fc3", 1024, 10))),
    3: Config(3, "encoder-d512", S=4, N=2048, dtype="bf16", r=10, iters=3,
              layers=(LayerShape("attn_proj", 512, 512, 4), LayerShape("ffn_up", 512, 2048),
                      LayerShape("ffn_down", 2048, 512))),
    4: Config(4, "vit-b", S=8, N=6304, dtype="bf16", r=16, iters=3, blocks=12,
              layers=(LayerShape("attn_proj", 768, 768, 4), LayerShape("ffn_up", 768, 3072),
                      LayerShape("ffn_down", 3072, 768))),
    5: Config(5, "gpt2-medium", S=16, N=4096, dtype="bf16", r=16, iters=3, blocks=24,
              layers=(LayerShape("attn_proj", 1024, 1024, 4), LayerShape("ffn_up", 1024, 4096),
                      LayerShape("ffn_down", 4096, 1024))),
}


def start_block(S: int, r: int, h_out: int, seed: int, device="cpu") -> torch.Tensor:
    """Random start vectors g_0 ~ N(0,1) of Algorithm 2, one r x h_out block per site (fp32)."""
    return torch.randn(S, r, h_out, generator=_gen(seed ^ 0x5EED, device), device=device, dtype=torch.float32)


def gaussian_layer(S: int, N: int, h_in: int, h_out: int, seed: int, dtype=torch.float32, device="cpu"):
    g = _gen(seed, device)
    A = torch.randn(S, N, h_in, generator=g, device=device, dtype=torch.float32)
    D = torch.randn(S, N, h_out, generator=g, device=device, dtype=torch.float32)
    return A.to(dtype).contiguous(), D.to(dtype).contiguous()


def decaying_layer(S: int, N: int, h_in: int, h_out: int, seed: int, dtype=torch.bfloat16, device="cpu",
                   modes: int = 64, noise: float = 0.02):
    """Activations ~ N(0,1); errors = (N(0,1) N x m) diag(1/k) (N(0,1) m x h_out)/sqrt(m) + noise,
    all scaled by 1/(S*N) as under a loss averaged over every sample of every site."""
    g = _gen(seed, device)
    m = max(1, min(modes, N, h_out))
    decay = 1.0 / torch.arange(1, m + 1, device=device, dtype=torch.float32)
    A = torch.empty(S, N, h_in, device=device, dtype=dtype)
    D = torch.empty(S, N, h_out, device=device, dtype=dtype)
    for s in range(S):
        A[s] = torch.randn(N, h_in, generator=g, device=device, dtype=torch.float32).to(dtype)
        U = torch.randn(N, m, generator=g, device=device, dtype=torch.float32) * decay
        V = torch.randn(m, h_out, generator=g, device=device, dtype=torch.float32) / (m ** 0.5)
        E = torch.randn(N, h_out, generator=g, device=device, dtype=torch.float32) * noise
        D[s] = ((U @ V + E) / float(S * N)).to(dtype)
    return A, D


# ------------------------------------------------------------------------------------------
# Config 2: ReLU MLP, softmax cross-entropy, float64 forward and backward by hand.
# ------------------------------------------------------------------------------------------
@dataclasses.dataclass
class MLPBatch:
    X: torch.Tensor          # S x N x h0 float64, U(0,1)
    labels: torch.Tensor     # S x N int64
    W: List[torch.Tensor]    # h_in x h_out float64 per layer (shared by every site)
    b: List[torch.Tensor]    # h_out float64 per layer
    A: List[torch.Tensor]    # per layer: S x N x h_in float64 (layer inputs)
    D: List[torch.Tensor]    # per layer: S x N x h_out float64 (errors at the layer's output)
    loss: float


def mlp_layers(S: int = 4, N: int = 128, sizes: Sequence[int] = (784, 1024, 1024, 10), seed: int = seed_for(2)) -> MLPBatch:
    """Forward Z_i = A_{i-1} W_i + B_i, A_i = relu(Z_i) (Eq. 1); loss = softmax cross-entropy
    averaged over all S*N samples; backward Delta_L = dL/dZ_L and
    Delta_i = (Delta_{i+1} W_{i+1}^T) * relu'(Z_i) (Sec. 3.1).  Every site holds the same
    weights (Sec. 3.3); all arithmetic in float64 on the CPU."""
    g = _gen(seed, "cpu")
    L = len(sizes) - 1
    X = torch.rand(S, N, sizes[0], generator=g, dtype=torch.float64)
    labels = torch.randint(0, sizes[-1], (S, N), generator=g)
    W, b = [], []
    for i in range(L):
        bound = 1.0 / (sizes[i] ** 0.5)
        W.append((torch.rand(sizes[i], sizes[i + 1], generator=g, dtype=torch.float64) * 2 - 1) * bound)
        b.append((torch.rand(sizes[i + 1], generator=g, dtype=torch.float64) * 2 - 1) * bound)
    acts = [X]
    pre = []
    for i in range(L):
        Z = acts[-1] @ W[i] + b[i]
        pre.append(Z)
        acts.append(torch.clamp_min(Z, 0.0) if i < L - 1 else Z)
    logits = pre[-1]
    m = logits.max(dim=-1, keepdim=True).values
    lse = m + torch.log(torch.exp(logits - m).sum(dim=-1, keepdim=True))
    logp = logits - lse
    onehot = torch.zeros_like(logits).scatter_(-1, labels.unsqueeze(-1), 1.0)
    loss = float(-(onehot * logp).sum() / (S * N))
    D = [None] * L
    D[L - 1] = (torch.exp(logp) - onehot) / float(S * N)
    for i in range(L - 2, -1, -1):
        D[i] = (D[i + 1] @ W[i + 1].T) * (pre[i] > 0).to(torch.float64)
    return MLPBatch(X=X, labels=labels, W=W, b=b, A=acts[:L], D=D, loss=loss)


# ------------------------------------------------------------------------------------------
# Config 3: one transformer encoder layer, forward/backward with hooks on its six linears.
# ------------------------------------------------------------------------------------------
class _EncoderLayer(torch.nn.Module):
    def __init__(self, d: int, heads: int, ffn: int):
        super().__init__()
        lin = torch.nn.Linear
        self.q, self.k, self.v, self.o = lin(d, d), lin(d, d), lin(d, d), lin(d, d)
        self.up, self.down = lin(d, ffn), lin(ffn, d)
        self.ln1, self.ln2 = torch.nn.LayerNorm(d), torch.nn.LayerNorm(d)
        self.heads = heads

    def forward(self, x):  # x: B x T x d
        B, T, d = x.shape
        H = self.heads
        y = self.ln1(x)
        q = self.q(y).view(B, T, H, d // H).transpose(1, 2)
        k = self.k(y).view(B, T, H, d // H).transpose(1, 2)
        v = self.v(y).view(B, T, H, d // H).transpose(1, 2)
        att = torch.softmax(q @ k.transpose(-1, -2) / ((d // H) ** 0.5), dim=-1)
        x = x + self.o((att @ v).transpose(1, 2).reshape(B, T, d))
        return x + self.down(torch.nn.functional.gelu(self.up(self.ln2(x))))


def encoder_layers(S: int = 4, batch: int = 16, seq: int = 128, d: int = 512, heads: int = 8, ffn: int = 2048,
                   seed: int = seed_for(3), dtype=torch.bfloat16):
    """Returns [(name, A, D)] for the projections q, k, v, o, up, down: A is S x (batch*seq) x h_in,
    D is S x (batch*seq) x h_out, cast to `dtype`.  Loss: mean over all sites' tokens of a random
    linear read-out, so D carries the 1/(S*N) of a global mean."""
    torch.manual_seed(seed)
    layer = _EncoderLayer(d, heads, ffn).float()
    names = ["q", "k", "v", "o", "up", "down"]
    mods = {n: getattr(layer, n) for n in names}
    cap_in = {n: [] for n in names}
    cap_out = {n: [] for n in names}
    hooks = []
    for n, m in mods.items():
        hooks.append(m.register_forward_hook(lambda mod, inp, out, n=n: cap_in[n].append(inp[0].detach())))
        hooks.append(m.register_full_backward_hook(lambda mod, gin, gout, n=n: cap_out[n].append(gout[0].detach())))
    g = _gen(seed + 1, "cpu")
    readout = torch.randn(d, generator=g)
    N = batch * seq
    for s in range(S):
        x = torch.randn(batch, seq, d, generator=g)
        loss = (layer(x) @ readout).sum() / float(S * N)
        loss.backward()
    for h in hooks:
        h.remove()
    out = []
    for n in names:
        A = torch.stack([t.reshape(N, -1) for t in cap_in[n]]).to(dtype).contiguous()
        D = torch.stack([t.reshape(N, -1) for t in cap_out[n]]).to(dtype).contiguous()
        out.append((n, A, D))
    return out


def layer_inputs(cfg: Config, shape: LayerShape, layer_index: int, device="cpu"):
    """(A, D, Q0) for one layer of a configuration, by the stand-in recipe of that configuration
    (config 1: plain N(0,1); otherwise the planted-spectrum recipe)."""
    seed = seed_for(cfg.index, layer_index)
    if cfg.index == 1:
        A, D = gaussian_layer(cfg.S, cfg.N, shape.h_in, shape.h_out, seed, cfg.torch_dtype, device)
    else:
        A, D = decaying_layer(cfg.S, cfg.N, shape.h_in, shape.h_out, seed, cfg.torch_dtype, device)
    Q0 = start_block(cfg.S, cfg.r, shape.h_out, seed, device)
    return A, D, Q0
