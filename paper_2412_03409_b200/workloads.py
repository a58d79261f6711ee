"""Seeded synthetic workloads (inputs only; none of the method's arithmetic).

The paper evaluates on LLaVA-1.5-7B/13B prompts (576 image tokens plus system
and instruction text, Sec. 4.1/4.3) whose weights and data are not available
here; these generators produce tensors of the same shapes with importance
concentration that differs by layer, as the paper's Fig. 3 observes.

One module serves both the CUDA library's tests and the CPU oracle's tests so
that both sides see the same bytes.  Tensors are created on the requested
device with a seeded ``torch.Generator``; a host copy of the same tensor is what
an oracle run consumes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    L: int
    H: int
    D: int
    N: int
    dtype: torch.dtype
    budget_ratios: tuple
    T: int                      # decode steps
    seed: int
    tol: float = 1e-6
    text_head: int = 0          # leading text positions (unit key scale)
    text_tail: int = 0          # trailing text positions
    layer_scale_mode: str = "loguniform"   # "fixed4" | "loguniform"
    key_bias: bool = False      # heavy-tailed per-key logit bias (Laplace)

    @property
    def esize(self) -> int:
        return 4 if self.dtype == torch.float32 else 2

    @property
    def row_bytes(self) -> int:
        return self.H * self.D * self.esize

    def budget_rows(self, ratio=None) -> int:
        r = self.budget_ratios[0] if ratio is None else ratio
        return int(math.floor(r * self.L * self.N + 1e-9))


WORKLOADS = {
    "tiny": Workload("tiny", 1, 4, 4, 64, 128, torch.float32, (0.5,), 16, seed=0,
                     layer_scale_mode="fixed4"),
    "llava7b_b1": Workload("llava7b_b1", 1, 32, 32, 128, 640, torch.bfloat16, (0.2,), 128,
                           seed=1, text_head=32, text_tail=32),
    "llava7b_b16": Workload("llava7b_b16", 16, 32, 32, 128, 640, torch.bfloat16,
                            (0.1, 0.2, 0.3, 0.5), 256, seed=2, text_head=32, text_tail=32),
    "llava13b_b8": Workload("llava13b_b8", 8, 40, 40, 128, 2048, torch.bfloat16, (0.2,), 512,
                            seed=3, text_head=64, text_tail=256),
    "longctx_b4": Workload("longctx_b4", 4, 32, 32, 128, 16384, torch.bfloat16, (0.05,), 1024,
                           seed=4, key_bias=True),
}
ORDER = ["tiny", "llava7b_b1", "llava7b_b16", "llava13b_b8", "longctx_b4"]
# A 4-sample cut of llava7b_b16, small enough (2 GB) for multi-pass profiler captures.
WORKLOADS["llava7b_b4"] = Workload("llava7b_b4", 4, 32, 32, 128, 640, torch.bfloat16, (0.2,), 64, seed=2,
                                   text_head=32, text_tail=32)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (reduced test cases)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


def layer_factors(w: Workload, b: int) -> np.ndarray:
    """Per-layer concentration factor s_l for sample b (host RNG, fp64)."""
    if w.layer_scale_mode == "fixed4":
        base = np.array([0.5, 1.0, 2.0, 4.0])
        return np.resize(base, w.L).astype(np.float64)
    rng = np.random.default_rng(w.seed * 7919 + 1000 * b + 17)
    return np.exp(rng.uniform(math.log(0.5), math.log(4.0), size=w.L))


def layer_scale(w: Workload) -> np.ndarray:
    """The scale[L] handed to the library: softmax logit = scale_l * <q, k>."""
    base = 1.0 / math.sqrt(w.D)
    if w.layer_scale_mode == "fixed4":
        return (layer_factors(w, 0) * base).astype(np.float32)
    return np.full(w.L, base, np.float32)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_prompt_sample(w: Workload, b: int, device="cpu"):
    """Q, K, V of one sample: each [L, H, N, D] in w.dtype on `device`."""
    g = _gen(device, w.seed * 1_000_003 + 1000 * b)
    shape = (w.L, w.H, w.N, w.D)
    out = []
    for name in ("q", "k", "v"):
        t = torch.empty(shape, dtype=torch.float32, device=device)
        # Per layer to bound the fp32 temporary at long prompts.
        for l in range(w.L):
            t[l].normal_(0.0, 1.0, generator=g)
        out.append(t)
    q, k, v = out
    if w.layer_scale_mode != "fixed4":
        s = torch.tensor(layer_factors(w, b), dtype=torch.float32, device=device)
        s = s.view(w.L, 1, 1, 1)
        if w.key_bias:
            # logit = scale * <q, k>_{D-1 dims} * s_l + bias_n: the bias rides on the
            # last channel (q = 1 there), the layer factor on the other channels.
            u = torch.rand((w.L, 1, w.N), generator=g, device=device) - 0.5
            bias = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
            k[..., : w.D - 1] *= s
            k[..., w.D - 1] = bias * math.sqrt(w.D)
            q[..., w.D - 1] = 1.0
        else:
            lo, hi = w.text_head, w.N - w.text_tail
            k[:, :, lo:hi, :] *= s
    return tuple(t.to(w.dtype) for t in (q, k, v))


def make_prompt(w: Workload, device="cpu", samples=None):
    """Q, K, V as [B', L, H, N, D] for the listed samples (default: all)."""
    samples = list(range(w.B)) if samples is None else list(samples)
    qs, ks, vs = [], [], []
    for b in samples:
        q, k, v = make_prompt_sample(w, b, device)
        qs.append(q); ks.append(k); vs.append(v)
    return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def make_decode_inputs(w: Workload, t: int, device="cpu", samples=None):
    """q, k_new, v_new of decode step t: each [B', L, H, D] in w.dtype."""
    samples = list(range(w.B)) if samples is None else list(samples)
    outs = [[], [], []]
    for b in samples:
        g = _gen(device, w.seed * 1_000_003 + 1000 * b + 7919 * (t + 1))
        for i in range(3):
            x = torch.empty((w.L, w.H, w.D), dtype=torch.float32, device=device)
            x.normal_(0.0, 1.0, generator=g)
            outs[i].append(x.to(w.dtype))
    return tuple(torch.stack(o) for o in outs)


def synthetic_scores(L: int, N: int, seed: int, concentration=None) -> np.ndarray:
    """Non-negative fp32 score rows with mean 1 and layer-dependent spread.

    Stands in for importance scores when only the selection stages are under
    test (no attention is computed).  Includes exact ties.
    """
    rng = np.random.default_rng(seed)
    conc = np.exp(rng.uniform(math.log(0.3), math.log(3.0), size=L)) if concentration is None \
        else np.asarray(concentration, dtype=np.float64)
    x = rng.standard_normal((L, N)) * conc[:, None]
    s = np.exp(x)
    s = s / s.mean(axis=1, keepdims=True)
    s = s.astype(np.float32)
    # plant ties: copy some values onto other positions
    n_ties = max(1, N // 16)
    for l in range(L):
        a = rng.integers(0, N, n_ties)
        b = rng.integers(0, N, n_ties)
        s[l, a] = s[l, b]
    return s
