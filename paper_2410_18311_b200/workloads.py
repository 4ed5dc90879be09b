"""Seeded synthetic inputs shaped like the models the method is evaluated on.

Only tensor shapes, seeds and random draws live here: none of the method's arithmetic
(no selection, no FFN).  The same tensors feed the CUDA path and the CPU oracle, so the
two sides always see identical bits; a tensor is generated once, on the device asked
for, and copied to the other side by the caller.

Seeds: 1000 * config id + layer for weights, + 500 for the prompt, + 700 + step for
decode inputs.  Weights ~ N(0, 0.02), prompt rows and decode inputs ~ N(0, 1), all cast
to the config's dtype; biases are absent (zero) unless a test adds them.
"""
from __future__ import annotations

import dataclasses

import torch


@dataclasses.dataclass(frozen=True)
class Config:
    cid: int
    name: str
    dtype: str            # "f32" | "bf16"
    gated: bool
    L: int
    d_model: int
    d_ff: int
    T: int
    alpha: float
    beta: float
    batch: int
    decode_steps: int
    planted: bool = False  # activations synthesised with a stable subset instead of a GEMM

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def esize(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def n_mat(self) -> int:
        return 3 if self.gated else 2

    def with_(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "opt125m-1layer": Config(1, "opt125m-1layer", "f32", False, 1, 768, 3072, 64, 0.4, 0.2, 1, 16),
    "opt6.7b": Config(2, "opt6.7b", "bf16", False, 32, 4096, 16384, 256, 0.4, 0.2, 1, 256),
    "opt13b": Config(3, "opt13b", "bf16", False, 40, 5120, 20480, 512, 0.4, 0.2, 1, 256),
    "relu-llama2-7b": Config(4, "relu-llama2-7b", "bf16", True, 32, 4096, 11008, 1024, 0.4, 0.25, 1, 256),
    "opt66b": Config(5, "opt66b", "bf16", False, 64, 9216, 36864, 512, 0.4, 0.2, 1, 128, planted=True),
}
# a seconds-scale stand-in with the same structure, for host-side tests of the harness
CONFIGS["tiny"] = Config(9, "tiny", "bf16", False, 2, 256, 1024, 16, 0.4, 0.2, 1, 4)
OPT13B_BETAS = (0.1, 0.2, 0.4, 1.0)
OPT66B_TS = (128, 512, 2048, 4096)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std, seed, device, dtype):
    t = torch.empty(shape, device=device, dtype=torch.float32)
    t.normal_(0.0, std, generator=_gen(seed, device))
    return t.to(dtype)


def layer_weights(cfg: Config, layer: int, device="cpu"):
    """(w_up [d_ff, d], w_gate [d_ff, d] | None, w_down [d, d_ff]) ~ N(0, 0.02) in cfg's dtype."""
    base = 1000 * cfg.cid + layer
    w_up = _normal((cfg.d_ff, cfg.d_model), 0.02, base * 16 + 1, device, cfg.torch_dtype)
    w_gate = _normal((cfg.d_ff, cfg.d_model), 0.02, base * 16 + 2, device, cfg.torch_dtype) if cfg.gated else None
    w_down = _normal((cfg.d_model, cfg.d_ff), 0.02, base * 16 + 3, device, cfg.torch_dtype)
    return w_up, w_gate, w_down


def compacted_weights_random(cfg: Config, layer: int, K: int, device="cpu"):
    """Random [K, d] buffers standing in for compacted weights of a layer (same distribution
    as a row/column subset of layer_weights): used where only the decode stage is exercised."""
    base = 1000 * cfg.cid + layer
    up = _normal((K, cfg.d_model), 0.02, base * 16 + 5, device, cfg.torch_dtype)
    gate = _normal((K, cfg.d_model), 0.02, base * 16 + 6, device, cfg.torch_dtype) if cfg.gated else None
    down = _normal((K, cfg.d_model), 0.02, base * 16 + 7, device, cfg.torch_dtype)
    return up, gate, down


def prompt_hidden(cfg: Config, device="cpu", T: int | None = None):
    """Prompt hidden states [T, d] ~ N(0, 1) (seed 0 for the one-layer fp32 config)."""
    seed = 0 if cfg.cid == 1 else 1000 * cfg.cid + 500
    return _normal((cfg.T if T is None else T, cfg.d_model), 1.0, seed, device, cfg.torch_dtype)


def decode_input(cfg: Config, step: int, device="cpu", batch: int | None = None):
    """Fresh decode-step input [batch, d] ~ N(0, 1)."""
    return _normal((cfg.batch if batch is None else batch, cfg.d_model), 1.0, 1000 * cfg.cid + 700 + step,
                   device, cfg.torch_dtype)


def planted_activations(cfg: Config, layer: int, T: int, device="cpu", sigma: float = 0.25):
    """Activations [T, d_ff] fp32 with the stability structure of Section 3.2: a fixed random
    15 % of the neurons draw Exp(1) in every row; every other entry is exactly 0 with
    probability 0.7 and |N(0, sigma)| otherwise.  Returns (A, planted_indices ascending)."""
    g = _gen(1000 * cfg.cid + 300 + layer, device)
    N = cfg.d_ff
    perm = torch.randperm(N, generator=g, device=device)
    n_core = int(0.15 * N)
    core = perm[:n_core].sort().values
    A = torch.empty((T, N), device=device, dtype=torch.float32)
    A.normal_(0.0, sigma, generator=g).abs_()
    keep = torch.rand((T, N), device=device, generator=g) >= 0.7
    A.mul_(keep)
    E = torch.empty((T, n_core), device=device, dtype=torch.float32)
    E.exponential_(1.0, generator=g)
    A[:, core] = E
    return A, core
