"""Seeded synthetic inputs: model shapes, random-init weights, prompts, schedules.

This module only draws numbers. It holds none of the method's arithmetic and is
the one piece shared by the CPU oracle's tests and the CUDA path's tests: both
sides are handed the very same arrays.

Stand-ins (no dataset or checkpoint is read):
  * weights: every matrix and the embedding ~ N(0, 0.02); RMSNorm gains = 1;
    LM head untied.  In bf16 mode every value is rounded once to bf16
    (round-to-nearest-even) at generation time, so both sides start from
    identical, bf16-representable numbers.
  * prompts: token ids uniform in [0, vocab).  Lengths follow the workload
    (3376 = mean prompt length of the long-context suite the paper evaluates on,
    Section 1 footnote; 4096; uniform 1024..4096 for the packed batch).
  * hidden states for the single-layer pruning op: N(0, 1).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Sequence, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4
    n_kv_heads: int = 0          # key/value heads; 0 = as many as query heads (no grouping)
    fp8: bool = False            # the four projections of a layer multiply e4m3 operands

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads or self.n_heads

    def with_kv_heads(self, n_kv_heads: int) -> "ModelShape":
        return dataclasses.replace(self, n_kv_heads=n_kv_heads)

    def with_fp8(self, on: bool = True) -> "ModelShape":
        return dataclasses.replace(self, fp8=on)

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers)


# Tiny fp32 decoder: 2 layers, d=256, 4 heads x 64, ffn 688, vocab 1024.
TINY = ModelShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=1024)
# Small bf16-friendly decoder with head_dim 128 for quick multi-tile parity cases.
SMALL = ModelShape(n_layers=4, d_model=512, n_heads=4, head_dim=128, d_ffn=1408, vocab=2048)
# Llama-2-7B shape (Section 1: 32 layers, model dimension 4096).
LLAMA7B = ModelShape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=32000)

# Cumulative keep 100/70/50/30 % entering layers 0/8/16/24, as (layer_entered, basis points).
SCHEDULE_7B: Tuple[Tuple[int, int], ...] = ((8, 7000), (16, 5000), (24, 3000))
SCHEDULE_TINY: Tuple[Tuple[int, int], ...] = ((1, 5000),)


def scaled_schedule(n_layers: int, schedule: Sequence[Tuple[int, int]] = SCHEDULE_7B,
                    ref_layers: int = 32) -> Tuple[Tuple[int, int], ...]:
    """The same keep fractions placed at the same relative depth of a shallower stack."""
    out = []
    for layer, bp in schedule:
        e = max(1, (layer * n_layers) // ref_layers)
        if out and e <= out[-1][0]:
            e = out[-1][0] + 1
        if e < n_layers:
            out.append((e, bp))
    return tuple(out)


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std: float, g: torch.Generator, device: str, bf16: bool) -> torch.Tensor:
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=g)
    if bf16:
        t = t.to(torch.bfloat16)
    return t


def make_weights(shape: ModelShape, seed: int, bf16: bool, device: str = "cpu",
                 std: float = 0.02) -> Dict[str, object]:
    """Random-init weights. Matrices are [out_features, in_features], row-major.

    Returned tensors are bf16 (if ``bf16``) or fp32.  Generation order is fixed,
    so a (shape, seed, device kind) triple always yields the same numbers.
    """
    g = _gen(seed, device)
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    dt = torch.bfloat16 if bf16 else torch.float32
    W: Dict[str, object] = {"tok_embed": _normal((V, d), std, g, device, bf16)}
    layers: List[Dict[str, torch.Tensor]] = []
    for _ in range(shape.n_layers):
        layers.append({
            "w_qkv": _normal((d + 2 * shape.kv_heads * shape.head_dim, d), std, g, device, bf16),
            "w_o": _normal((d, d), std, g, device, bf16),
            "w_gate": _normal((F, d), std, g, device, bf16),
            "w_up": _normal((F, d), std, g, device, bf16),
            "w_down": _normal((d, F), std, g, device, bf16),
            "g_attn": torch.ones(d, dtype=dt, device=device),
            "g_mlp": torch.ones(d, dtype=dt, device=device),
        })
    W["layers"] = layers
    W["g_final"] = torch.ones(d, dtype=dt, device=device)
    W["w_lm_head"] = _normal((V, d), std, g, device, bf16)
    return W


def perturb_gains(W: Dict[str, object], seed: int) -> None:
    """Replace the unit RMSNorm gains by 1 + 0.1*N(0,1) (tests only: a unit gain hides
    a forgotten or misplaced gain multiply)."""
    g = _gen(seed, "cpu")
    def p(t: torch.Tensor) -> torch.Tensor:
        r = torch.empty(t.shape, dtype=torch.float32).normal_(0.0, 0.1, generator=g)
        return (1.0 + r).to(t.dtype).to(t.device)
    for lw in W["layers"]:
        lw["g_attn"] = p(lw["g_attn"])
        lw["g_mlp"] = p(lw["g_mlp"])
    W["g_final"] = p(W["g_final"])


def make_prompt(vocab: int, n_tokens: int, seed: int, device: str = "cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randint(0, vocab, (n_tokens,), generator=g, device=device, dtype=torch.int32)


def make_varlen_lengths(n_seqs: int, lo: int, hi: int, seed: int) -> List[int]:
    """Sequence lengths uniform in [lo, hi] (inclusive)."""
    g = _gen(seed, "cpu")
    return [int(v) for v in torch.randint(lo, hi + 1, (n_seqs,), generator=g)]


def make_varlen_batch(vocab: int, lengths: Sequence[int], seed: int,
                      device: str = "cpu") -> Tuple[torch.Tensor, List[int]]:
    """Packed ids and cu_seqlens for a batch of independent prompts."""
    ids = make_prompt(vocab, int(sum(lengths)), seed, device)
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + int(n))
    return ids, cu


def make_hidden(n_rows: int, d_model: int, seed: int, bf16: bool,
                device: str = "cpu") -> torch.Tensor:
    """Hidden states ~ N(0,1) for the single-layer pruning op."""
    return _normal((n_rows, d_model), 1.0, _gen(seed, device), device, bf16)


def make_scores(n: int, kind: str, seed: int) -> torch.Tensor:
    """Score vectors for the selection stress cases (fp32, non-negative)."""
    g = _gen(seed, "cpu")
    if kind == "uniform":
        return torch.full((n,), 1.0 / n, dtype=torch.float32)
    if kind == "lognormal":
        s = torch.empty(n, dtype=torch.float32).log_normal_(0.0, 2.0, generator=g)
        return s / s.sum()
    if kind == "zeros":
        s = torch.rand(n, generator=g, dtype=torch.float32)
        s[torch.rand(n, generator=g) < 0.7] = 0.0
        return s
    if kind == "duplicates":
        levels = torch.tensor([0.0, 0.125, 0.25, 0.5], dtype=torch.float32)
        return levels[torch.randint(0, 4, (n,), generator=g)]
    if kind == "random":
        return torch.rand(n, generator=g, dtype=torch.float32)
    raise ValueError(kind)


PROJECTIONS = ("w_qkv", "w_o", "w_gate", "w_up", "w_down")


def quantize_projections_e4m3(W: Dict[str, object]) -> Dict[str, object]:
    """8-bit copies of the projection matrices of every layer: per matrix a power-of-two scale >= max|w| / 448
    and the e4m3 codes of w / scale (torch's float8_e4m3fn cast: round to nearest even).  The bf16 / fp32
    matrices in W are REPLACED by their de-quantised values codes * scale, which a power-of-two scale makes
    exactly representable in bf16 (four significant bits), so the 8-bit path, the bf16 path and the oracle
    all see the very same weights.  Returns {"layers": [{name: (codes as uint8, scale)}]}."""
    out = {"layers": []}
    for lw in W["layers"]:
        q = {}
        for name in PROJECTIONS:
            w = lw[name].float()
            amax = float(w.abs().max())
            scale = 2.0 ** math.ceil(math.log2(amax / 448.0)) if amax > 0 else 1.0
            codes = (w / scale).to(torch.float8_e4m3fn)
            q[name] = (codes.view(torch.uint8), scale)
            lw[name] = (codes.float() * scale).to(lw[name].dtype)
        out["layers"].append(q)
    return out
