"""Seeded synthetic workloads: weight matrices and calibration activations.

This module only makes inputs.  It holds none of the pruning method's
arithmetic, so that both the CUDA library's tests and the CPU oracle's tests
can be fed from it without sharing anything else.

The workloads have the linear-layer shapes of the model families the paper
prunes (Section 4.1: Pythia, LLaMA-2, LLaMA-3) with i.i.d. N(0, 0.02^2) weights
and calibration activations whose bulk is Gaussian or Student-t(3) and in which
a small set of seeded "outlier" input channels is scaled up, which is the
structure LLM activations are known to have.  Every tensor is a pure function
of (workload name, block, tensor name, batch index) and the base seed.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field

import torch

FP16_CLAMP = 60000.0  # heavy tails times the outlier scale would overflow binary16


@dataclass(frozen=True)
class LayerSpec:
    name: str      # e.g. "q_proj"
    d_out: int     # rows of W
    d_in: int      # columns of W = width of the input it reads
    input: str     # which calibration input it reads ("attn_in", "o_in", "mlp_in", "down_in")


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                 # "f16" | "bf16"
    blocks: int
    layers: tuple              # LayerSpec per block
    n_seqs: int
    seq_len: int
    x_dist: str                # "normal" | "student_t3" | "student_t3_chanscale"
    outlier_frac: float = 0.0  # fraction of channels scaled by outlier_scale
    n_outliers: int = -1       # overrides outlier_frac when >= 0
    outlier_scale: float = 20.0
    mode: str = "unstructured"  # "unstructured" | "nm"
    sparsities: tuple = (0.5,)
    patterns: tuple = ()        # ((N, M), ...) for mode "nm"
    passes: int = 1             # repeated-prune loop length
    seed: int = 0
    inputs: dict = field(default_factory=dict, compare=False)

    @property
    def tokens(self) -> int:
        return self.n_seqs * self.seq_len

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "f16" else torch.bfloat16

    def input_widths(self) -> dict:
        w = {}
        for l in self.layers:
            w.setdefault(l.input, l.d_in)
        return w

    def weights_per_block(self) -> int:
        return sum(l.d_out * l.d_in for l in self.layers)

    def total_weights(self) -> int:
        return self.blocks * self.weights_per_block()


def _llama_layers(d, d_ff, d_kv=None):
    d_kv = d if d_kv is None else d_kv
    return (
        LayerSpec("q_proj", d, d, "attn_in"),
        LayerSpec("k_proj", d_kv, d, "attn_in"),
        LayerSpec("v_proj", d_kv, d, "attn_in"),
        LayerSpec("o_proj", d, d, "o_in"),
        LayerSpec("gate_proj", d_ff, d, "mlp_in"),
        LayerSpec("up_proj", d_ff, d, "mlp_in"),
        LayerSpec("down_proj", d, d_ff, "down_in"),
    )


WORKLOADS = {
    # one small layer: the case the CPU oracle finishes in well under a second
    "single-512": Workload(
        "single-512", "f16", 1, (LayerSpec("linear", 512, 512, "in"),),
        n_seqs=16, seq_len=128, x_dist="normal", n_outliers=4, mode="unstructured",
        sparsities=(0.5,)),
    "pythia-410m": Workload(
        "pythia-410m", "f16", 24,
        (LayerSpec("qkv", 3072, 1024, "attn_in"), LayerSpec("attn_out", 1024, 1024, "o_in"),
         LayerSpec("mlp_up", 4096, 1024, "mlp_in"), LayerSpec("mlp_down", 1024, 4096, "down_in")),
        n_seqs=128, seq_len=512, x_dist="normal", outlier_frac=0.005, mode="unstructured",
        sparsities=(0.5,)),
    "llama2-7b": Workload(
        "llama2-7b", "f16", 32, _llama_layers(4096, 11008),
        n_seqs=128, seq_len=2048, x_dist="student_t3", outlier_frac=0.005, mode="nm",
        patterns=((2, 4),)),
    "llama3-8b": Workload(
        "llama3-8b", "bf16", 32, _llama_layers(4096, 14336, 1024),
        n_seqs=128, seq_len=2048, x_dist="student_t3_chanscale", mode="unstructured",
        sparsities=(0.5, 0.6, 0.7, 0.8)),
    "llama2-13b": Workload(
        "llama2-13b", "f16", 40, _llama_layers(5120, 13824),
        n_seqs=128, seq_len=2048, x_dist="student_t3", outlier_frac=0.005, mode="nm",
        patterns=((2, 4), (4, 8)), passes=10),
}


def scaled(w: Workload, *, blocks=None, n_seqs=None, seq_len=None, shrink=1) -> Workload:
    """A smaller workload of the same family (for tests): fewer blocks/tokens and
    every layer dimension divided by ``shrink``."""
    layers = tuple(LayerSpec(l.name, max(8, l.d_out // shrink), max(8, l.d_in // shrink), l.input)
                   for l in w.layers)
    return Workload(w.name + "-scaled", w.dtype, blocks or w.blocks, layers,
                    n_seqs or w.n_seqs, seq_len or w.seq_len, w.x_dist, w.outlier_frac,
                    w.n_outliers, w.outlier_scale, w.mode, w.sparsities, w.patterns, w.passes,
                    w.seed)


def tensor_seed(base_seed: int, *key) -> int:
    """Stable 63-bit seed from a base seed and a tuple of names/indices."""
    h = hashlib.blake2b(repr((base_seed,) + key).encode(), digest_size=8).digest()
    return int.from_bytes(h, "little") & 0x7FFFFFFFFFFFFFFF


def _generator(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def gen_weight(w: Workload, block: int, layer: LayerSpec, device="cpu") -> torch.Tensor:
    """W [d_out, d_in] ~ N(0, 0.02^2), rounded to the workload's 16-bit type."""
    g = _generator(device, tensor_seed(w.seed, w.name, block, layer.name, "W"))
    t = torch.empty(layer.d_out, layer.d_in, dtype=torch.float32, device=device)
    t.normal_(0.0, 0.02, generator=g)
    return t.to(w.torch_dtype)


def outlier_channels(w: Workload, block: int, input_name: str, d_in: int) -> torch.Tensor:
    """Indices (sorted, on CPU) of the channels that get the outlier scale."""
    k = w.n_outliers if w.n_outliers >= 0 else int(round(w.outlier_frac * d_in))
    if k <= 0:
        return torch.empty(0, dtype=torch.long)
    g = _generator("cpu", tensor_seed(w.seed, w.name, block, input_name, "outlier-idx"))
    return torch.randperm(d_in, generator=g)[:k].sort().values


def channel_scale(w: Workload, block: int, input_name: str, d_in: int) -> torch.Tensor:
    """Per-channel multiplier [d_in] (float32, CPU) applied to the bulk distribution."""
    s = torch.ones(d_in, dtype=torch.float32)
    if w.x_dist == "student_t3_chanscale":
        g = _generator("cpu", tensor_seed(w.seed, w.name, block, input_name, "chan-scale"))
        z = torch.empty(d_in, dtype=torch.float32).normal_(0.0, 1.0, generator=g)
        s = torch.exp(z).clamp_(max=50.0)
    idx = outlier_channels(w, block, input_name, d_in)
    if idx.numel():
        s[idx] *= w.outlier_scale
    return s


def gen_activations(w: Workload, block: int, input_name: str, d_in: int, seq_begin: int,
                    n_seqs: int, device="cpu", out: torch.Tensor | None = None) -> torch.Tensor:
    """Calibration activations of sequences [seq_begin, seq_begin + n_seqs):
    a [n_seqs * seq_len, d_in] tensor in the workload's 16-bit type.  Each sequence
    has its own seed, so any batching of the sequences gives the same numbers."""
    scale = channel_scale(w, block, input_name, d_in).to(device)
    T = n_seqs * w.seq_len
    if out is None:
        out = torch.empty(T, d_in, dtype=w.torch_dtype, device=device)
    for s in range(n_seqs):
        g = _generator(device, tensor_seed(w.seed, w.name, block, input_name, "X", seq_begin + s))
        z = torch.empty(w.seq_len, d_in, dtype=torch.float32, device=device)
        z.normal_(0.0, 1.0, generator=g)
        if w.x_dist.startswith("student_t3"):
            # t(3) = N(0,1) / sqrt(chi2(3) / 3)
            chi = torch.zeros_like(z)
            for _ in range(3):
                u = torch.empty_like(z).normal_(0.0, 1.0, generator=g)
                chi.addcmul_(u, u)
            z.div_(chi.div_(3.0).sqrt_())
        z.mul_(scale)
        z.clamp_(-FP16_CLAMP, FP16_CLAMP)
        out[s * w.seq_len:(s + 1) * w.seq_len].copy_(z)
    return out


def bits_of(t: torch.Tensor):
    """uint16 numpy view of a CPU 16-bit float tensor's bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
