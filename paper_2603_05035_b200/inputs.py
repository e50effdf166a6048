"""Seeded synthetic inputs for the GELO Q/K/V offload path.

This module holds no arithmetic of the method: it only draws the hidden states
``H`` and the fused projection weight ``W_qkv`` with the shapes and value
distributions of Llama-2-7B attention layers and rounds them ONCE to the path's
storage type.  The CUDA library and the test oracle both consume exactly these
bytes.

Recipe (stands in for real Llama-2-7B activations and weights, which are not
available offline):

* ``H``  : n x d, i.i.d. N(0, 1); with ``rms_norm`` every row is divided by its
  root-mean-square so that all row norms equal sqrt(d) (a pre-attention RMSNorm
  without learned gain).
* ``W``  : d x p with p = 3 d, i.i.d. N(0, 0.02^2), columns ordered [W_q | W_k | W_v].
* dtype : "f32", "bf16" or "f16" (round-to-nearest-even from fp32, once).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

ORTHOGONAL = 0
NONORTHOGONAL = 1


@dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration of the offload path."""
    name: str
    n: int            # data token rows per call
    k: int            # shield rows per call
    d: int            # model width
    p: int            # fused projection width (3 d)
    dtype: str        # "f32" | "bf16"
    kinds: tuple      # mixing kind per call, cycled over calls
    shield_scale: float
    rms_norm: bool
    seed: int
    calls: int        # projection calls in one sweep (layers)

    @property
    def m(self) -> int:
        return self.n + self.k

    def kind(self, call: int) -> int:
        return self.kinds[call % len(self.kinds)]


WORKLOADS = {
    # tiny fp32 correctness case: orthogonal A, no shields
    "tiny_f32": Workload("tiny_f32", 64, 0, 256, 768, "f32", (ORTHOGONAL,), 0.0, False, 0, 1),
    # one Llama-2-7B-shaped layer in fp32, non-orthogonal A, no shields
    "layer_f32": Workload("layer_f32", 512, 0, 4096, 12288, "f32", (NONORTHOGONAL,), 0.0, True, 1, 1),
    # bf16 operands, orthogonal A, 5% shield rows at 10x the median row norm
    "shield_bf16": Workload("shield_bf16", 2048, 102, 4096, 12288, "bf16", (ORTHOGONAL,), 10.0, True, 2, 1),
    # prefill sweep over 32 layers, 4 sequences x 1024 tokens, alternating mixing kinds
    "prefill_bf16": Workload("prefill_bf16", 4096, 204, 4096, 12288, "bf16",
                             (ORTHOGONAL, NONORTHOGONAL), 10.0, True, 3, 32),
    # decode-shaped: 64 sequences x 1 token, 4 shield rows
    "decode_bf16": Workload("decode_bf16", 64, 4, 4096, 12288, "bf16", (ORTHOGONAL,), 10.0, True, 4, 32),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[name]


def _generator(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_hidden(n: int, d: int, dtype: str, seed: int, rms_norm: bool, device="cpu") -> torch.Tensor:
    """n x d hidden states in the storage dtype."""
    g = _generator(device, 2 * int(seed) + 1)
    h = torch.randn((n, d), generator=g, device=device, dtype=torch.float32)
    if rms_norm:
        h = h / torch.sqrt(torch.mean(h * h, dim=1, keepdim=True))
    return h.to(torch_dtype(dtype)).contiguous()


def make_weight(d: int, p: int, dtype: str, seed: int, device="cpu") -> torch.Tensor:
    """d x p fused projection weight [W_q | W_k | W_v] in the storage dtype."""
    g = _generator(device, 2 * int(seed) + 2)
    w = torch.randn((d, p), generator=g, device=device, dtype=torch.float32) * 0.02
    return w.to(torch_dtype(dtype)).contiguous()


def make_call_inputs(w: Workload, call: int = 0, device="cpu"):
    """(H, W, seed) of projection call ``call`` of workload ``w``.

    The returned seed is the one handed to the mixing sampler for that call, so
    every call draws a fresh A.
    """
    seed = w.seed + call
    h = make_hidden(w.n, w.d, w.dtype, seed, w.rms_norm, device)
    wt = make_weight(w.d, w.p, w.dtype, seed, device)
    return h, wt, seed


def to_f64_numpy(t: torch.Tensor):
    """Exact widening of a stored tensor to a float64 numpy array (for the oracle)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
