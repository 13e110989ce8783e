"""Seeded synthetic workloads: tensor lists, initial state and gradients.

This module only *produces inputs*.  It contains none of the optimizer's
arithmetic (no Adam update, no norm/clip decision, no rounding rule of the
method) and imports neither the CUDA binding nor the CPU oracle, so both can
be fed the same bits.  Tensor lists are shaped like the transformer models the
paper trains (GPT/LLaMA-style stacks, Section 5.1 and Appendix A); values are
random stand-ins, since the optimizer step is data-oblivious.

Value recipe (all workloads):  master weights ~ N(0, 0.02) in fp32, first and
second moments zero, gradients ~ N(0, sigma_g) rounded to bf16 by torch's own
conversion (or kept fp32), one fresh draw per step from
``torch.Generator(seed = base_seed * 1_000_003 + step)``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Tuple

import torch

MI = 1 << 20


@dataclass(frozen=True)
class Fault:
    """A non-finite value written into the gradient of one step."""
    step: int            # 1-based iteration
    flat_index: int      # position in the flat parameter space
    kind: str            # "inf" | "-inf" | "nan"


@dataclass
class Workload:
    name: str
    numel: List[int]                 # one entry per tensor, flattening order
    bucket_elems: int
    sigma_g: float = 1e-3
    sigma_p: float = 0.02
    steps: int = 10
    seed: int = 0
    max_grad_norm: float = 1.0       # <= 0: clipping off
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    grad_dtype: str = "bf16"         # "bf16" | "fp32" | "fp16"
    # fp16 gradients are stored multiplied by a loss scale (initial value and
    # dynamic schedule: growth / backoff factors, clean iterations before growth)
    loss_scale: float = 1.0
    ls_growth: float = 2.0
    ls_backoff: float = 0.5
    ls_interval: int = 0
    faults: Tuple[Fault, ...] = ()
    # optional: target global gradient norm per step (gradients are rescaled)
    target_norm: Optional[Callable[[int], float]] = None
    # optional: periodic NaN (every k-th step) at a seeded position
    nan_every: int = 0
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def total(self) -> int:
        return sum(self.numel)

    @property
    def n_buckets(self) -> int:
        return -(-self.total // self.bucket_elems)


# --------------------------------------------------------------------------
# tensor lists
# --------------------------------------------------------------------------

def gpt2_small_numel() -> List[int]:
    """GPT-2-small-shaped list: 12 layers, d=768, ffn 3072, vocab 50257."""
    d, ffn, vocab, ctx, layers = 768, 3072, 50257, 1024, 12
    out = [vocab * d, ctx * d]
    for _ in range(layers):
        out += [d, d,                 # ln_1 weight, bias
                d * 3 * d, 3 * d,     # fused qkv
                d * d, d,             # attention projection
                d, d,                 # ln_2
                d * ffn, ffn,         # mlp up
                ffn * d, d]           # mlp down
    out += [d, d]                     # final layer norm
    return out


def _llama_numel(layers, d, ffn, n_q, n_kv, vocab, tied_head) -> List[int]:
    head = d // n_q
    kv = n_kv * head
    out = [vocab * d]
    if not tied_head:
        out.append(vocab * d)
    for _ in range(layers):
        out += [d * d, d * kv, d * kv, d * d,      # q, k, v, o
                d * ffn, d * ffn, ffn * d,         # gate, up, down
                d, d]                              # two RMS norms
    out.append(d)                                  # final norm
    return out


def llama_1b_numel() -> List[int]:
    """Llama-3.2-1B-shaped: 16 layers, d=2048, ffn 8192, 32q/8kv, tied head."""
    return _llama_numel(16, 2048, 8192, 32, 8, 128256, tied_head=True)


def llama_8b_numel() -> List[int]:
    """Llama-3-8B-shaped: 32 layers, d=4096, ffn 14336, 32q/8kv, separate head."""
    return _llama_numel(32, 4096, 14336, 32, 8, 128256, tied_head=False)


# --------------------------------------------------------------------------
# the benchmark configurations
# --------------------------------------------------------------------------

def tiny() -> Workload:
    """1 Mi parameters in 4 buckets; every step clips; +inf on step 7."""
    return Workload(name="tiny", numel=[MI], bucket_elems=262_144, sigma_g=1e-2, steps=10,
                    faults=(Fault(step=7, flat_index=2 * 262_144 + 131_072, kind="inf"),),
                    notes="clip=1.0 < norm ~ 10.24: CLIP_RESTEP every step, SKIP on step 7")


def tiny_fp16() -> Workload:
    """The tiny case with fp16 gradients under dynamic loss scaling: the
    initial scale overflows fp16, so the first iterations are skipped while the
    scale backs off; afterwards it grows every 3 clean iterations until it
    overflows again."""
    w = tiny()
    w.name = "tiny_fp16"
    w.grad_dtype = "fp16"
    w.faults = ()
    w.loss_scale = 2.0 ** 23
    w.ls_interval = 3
    return w


def tiny_ragged() -> Workload:
    """The tiny case cut into odd-sized tensors and an odd bucket size."""
    sizes = [1, 7, 262_143, 5, 100_003, 333_331, 64, 2, 352_020]
    w = tiny()
    w.name = "tiny_ragged"
    w.numel = sizes
    w.bucket_elems = 250_003
    w.faults = (Fault(step=7, flat_index=2 * 250_003 + 17, kind="inf"),)
    return w


def gpt2_small(clip: bool = False) -> Workload:
    return Workload(name="gpt2_small_clip" if clip else "gpt2_small", numel=gpt2_small_numel(),
                    bucket_elems=25_000_000, sigma_g=1e-3, steps=20,
                    max_grad_norm=1.0 if clip else 0.0,
                    notes="124M parameters, 5 buckets of 25M (last partial)")


def llama_1b() -> Workload:
    return Workload(name="llama_1b", numel=llama_1b_numel(), bucket_elems=100_000_000,
                    sigma_g=1.0, steps=100, max_grad_norm=1.0,
                    target_norm=lambda step: 0.5 if step % 2 == 1 else 3.0, nan_every=50,
                    notes="global norm alternates 0.5 / 3.0; NaN every 50 steps")


def llama_8b() -> Workload:
    return Workload(name="llama_8b", numel=llama_8b_numel(), bucket_elems=200_000_000,
                    sigma_g=5e-6, steps=10, max_grad_norm=1.0,
                    notes="norm ~ 0.45 < clip: COMMIT every step")


def sweep(bucket_mi: int, grad_dtype: str = "bf16", total: int = 4 << 30) -> Workload:
    return Workload(name=f"sweep_{bucket_mi}Mi_{grad_dtype}", numel=[total],
                    bucket_elems=bucket_mi * MI, sigma_g=1e-3, steps=10, max_grad_norm=0.0,
                    grad_dtype=grad_dtype, loss_scale=4096.0 if grad_dtype == "fp16" else 1.0)


def _with_grad_dtype(w: Workload, dtype: str) -> Workload:
    """The same list with fp32 gradients, or fp16 gradients under a static loss scale."""
    w.name = f"{w.name}_{dtype}"
    w.grad_dtype = dtype
    if dtype == "fp16":
        w.loss_scale = 4096.0
    return w


def by_name(name: str) -> Workload:
    table = {"tiny": tiny, "tiny_ragged": tiny_ragged, "tiny_fp16": tiny_fp16,
             "gpt2_small": gpt2_small,
             "gpt2_small_clip": lambda: gpt2_small(clip=True),
             "gpt2_small_fp32": lambda: _with_grad_dtype(gpt2_small(), "fp32"),
             "gpt2_small_fp16": lambda: _with_grad_dtype(gpt2_small(), "fp16"),
             "llama_1b": llama_1b, "llama_8b": llama_8b}
    if name in table:
        return table[name]()
    if name.startswith("sweep_"):
        _, mi, dt = name.split("_")
        return sweep(int(mi.rstrip("Mi")), dt)
    raise KeyError(name)


# --------------------------------------------------------------------------
# value generators (seeded, device-agnostic)
# --------------------------------------------------------------------------

def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def iter_initial_master(w: Workload, device="cpu", chunk: int = 1 << 26):
    """Yields (start, fp32 tensor) pieces of the flat master weights in order.
    The pieces are drawn from one generator, so the values do not depend on
    who consumes them (a flat tensor or the slot arenas directly)."""
    gen = _gen(device, w.seed * 1_000_003 + 999_983)
    for s in range(0, w.total, chunk):
        e = min(s + chunk, w.total)
        z = torch.empty(e - s, dtype=torch.float32, device=device)
        z.normal_(0.0, w.sigma_p, generator=gen)
        yield s, z


def initial_master(w: Workload, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """Flat fp32 master weights ~ N(0, sigma_p), seeded by the workload."""
    out = torch.empty(w.total, dtype=torch.float32, device=device)
    for s, z in iter_initial_master(w, device, chunk):
        out[s:s + z.numel()] = z
    return out


def _fault_value(kind: str) -> float:
    return {"inf": float("inf"), "-inf": float("-inf"), "nan": float("nan")}[kind]


def faults_for_step(w: Workload, step: int) -> List[Fault]:
    """Faults injected into the gradient of iteration ``step`` (1-based)."""
    out = [f for f in w.faults if f.step == step]
    if w.nan_every and step % w.nan_every == 0:
        pos = _gen("cpu", w.seed * 7_919 + step)
        idx = int(torch.randint(0, w.total, (1,), generator=pos).item())
        out.append(Fault(step=step, flat_index=idx, kind="nan"))
    return out


_TORCH_DTYPE = {"bf16": torch.bfloat16, "fp32": torch.float32, "fp16": torch.float16}


def iter_gradients(w: Workload, step: int, device="cpu", chunk: int = 1 << 26,
                   loss_scale: float = 1.0):
    """Yields (start, tensor) pieces of the flat gradient of iteration ``step``
    (1-based) in order, in the workload's gradient dtype.

    Drawn in fp32 ~ N(0, sigma_g); when the workload fixes a target global
    norm the draw is rescaled by ``target / ||draw||`` (double precision
    scalar) before the rounding to the gradient dtype; ``loss_scale`` (fp16
    training) multiplies the value that gets stored, so large scales overflow
    to infinity exactly as a scaled backward pass would; faults are written last.
    """
    dtype = _TORCH_DTYPE[w.grad_dtype]
    gen = _gen(device, w.seed * 1_000_003 + step)
    scale = None
    if w.target_norm is not None:
        # first pass: norm of the fp32 draw; the second pass re-draws the same bits
        acc = 0.0
        state = gen.get_state()
        for s in range(0, w.total, chunk):
            e = min(s + chunk, w.total)
            z = torch.empty(e - s, dtype=torch.float32, device=device)
            z.normal_(0.0, w.sigma_g, generator=gen)
            acc += float(z.double().pow(2).sum().item())
        gen.set_state(state)
        scale = w.target_norm(step) / (acc ** 0.5)
    faults = faults_for_step(w, step)
    for s in range(0, w.total, chunk):
        e = min(s + chunk, w.total)
        z = torch.empty(e - s, dtype=torch.float32, device=device)
        z.normal_(0.0, w.sigma_g, generator=gen)
        if scale is not None:
            z = (z.double() * scale).float()
        if loss_scale != 1.0:
            z = z * loss_scale
        z = z.to(dtype)
        for f in faults:
            if s <= f.flat_index < e:
                z[f.flat_index - s] = _fault_value(f.kind)
        yield s, z


def gradients(w: Workload, step: int, device="cpu", chunk: int = 1 << 26,
              loss_scale: float = 1.0) -> torch.Tensor:
    """Flat gradient of iteration ``step`` (1-based) in the workload's dtype."""
    out = torch.empty(w.total, dtype=_TORCH_DTYPE[w.grad_dtype], device=device)
    for s, z in iter_gradients(w, step, device, chunk, loss_scale):
        out[s:s + z.numel()] = z
    return out


def bf16_bits(t: torch.Tensor) -> torch.Tensor:
    """Reinterpret a bf16 tensor as its int16 bit patterns (no arithmetic)."""
    return t.view(torch.int16)
