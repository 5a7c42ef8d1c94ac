"""Seeded synthetic replica sets for the five benchmark workloads.

This module only *generates inputs*: tensor shapes, value distributions and
fault patches.  It holds none of the sign/vote arithmetic and is the one piece
both the CUDA path's tests and the CPU oracle's tests may import.  It needs
torch for random numbers and device memory, nothing else.

The workloads stand in for what the paper checks with exact consensus: layer
outputs, gradient buckets, updated weights and optimizer slots (Sec. 5.2,
Sec. 9 "Optimizer boundary").  No dataset is involved.

Recipe (seed S = 0x5C0070000 + 16*config + case):
  * values come from ``torch.Generator(device).manual_seed(S)``; every replica
    is a byte-for-byte copy of replica 0;
  * faults come from ``random.Random(S + 1)`` as a list of patches
    (replica, tensor, element, operation on the element's integer pattern).
"""
from __future__ import annotations

import math
import random
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

SEED_BASE = 0x5C0070000

DTYPE_BYTES = {"u8": 1, "f32": 4, "bf16": 2, "i64": 8, "f16": 2, "f64": 8, "i32": 4}
TORCH_DTYPE = {"u8": torch.uint8, "f32": torch.float32, "bf16": torch.bfloat16,
               "i64": torch.int64, "f16": torch.float16, "f64": torch.float64,
               "i32": torch.int32}
INT_VIEW = {1: torch.uint8, 2: torch.int16, 4: torch.int32, 8: torch.int64}


@dataclass
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    dtype: str                  # key of DTYPE_BYTES
    dist: str                   # "normal" | "absnormal" | "randint40" | "randfull" | "bytes"
    std: float = 1.0

    @property
    def numel(self) -> int:
        return int(math.prod(self.shape))

    @property
    def nbytes(self) -> int:
        return self.numel * DTYPE_BYTES[self.dtype]


@dataclass
class Patch:
    replica: int
    tensor: int
    element: int
    op: str                     # "xor" | "set" | "add" on the element's integer pattern
    value: int


@dataclass
class Workload:
    name: str
    config: int
    case: str
    R: int
    chunk_bytes: int
    specs: List[TensorSpec]
    seed: int
    patches: List[Patch] = field(default_factory=list)
    # chunk-local groups that must come out without a strict majority
    note: str = ""

    @property
    def bytes_per_replica(self) -> int:
        return sum(s.nbytes for s in self.specs)


def seed_for(config: int, case_index: int = 0) -> int:
    return SEED_BASE + 16 * config + case_index


# ---------------------------------------------------------------- tensor lists

def _cfg3_specs(layers: int, d_model: int, d_ff: int) -> List[TensorSpec]:
    specs = []
    for l in range(layers):
        for i in range(4):
            specs.append(TensorSpec(f"l{l}.attn{i}", (d_model, d_model), "bf16", "normal", 0.02))
        for i in range(2):
            specs.append(TensorSpec(f"l{l}.up{i}", (d_ff, d_model), "bf16", "normal", 0.02))
        specs.append(TensorSpec(f"l{l}.down", (d_model, d_ff), "bf16", "normal", 0.02))
    return specs


def _cfg5_specs(n_tensors: int, lo: int, hi: int, rng: random.Random) -> List[TensorSpec]:
    """Sizes log-uniform in [lo, hi] bytes, rounded down to a multiple of 8."""
    specs = []
    for i in range(n_tensors):
        size = int(math.exp(rng.uniform(math.log(lo), math.log(hi))))
        size = max(8, size - size % 8)
        dt = rng.choice(["f32", "bf16", "i64"])
        numel = size // DTYPE_BYTES[dt]
        if dt == "i64":
            specs.append(TensorSpec(f"t{i}", (numel,), dt, "randint40"))
        else:
            specs.append(TensorSpec(f"t{i}", (numel,), dt, "normal", 0.02))
    return specs


def _int_bits(dtype: str) -> int:
    return 8 * DTYPE_BYTES[dtype]


def workload(config: int, case: str = "default", scale: float = 1.0) -> Workload:
    """The five benchmark workloads.  ``scale`` < 1 shrinks element counts
    (same R, dtypes, chunk size and fault recipe) for quick tests."""
    case_index = {"default": 0, "clean": 0, "mantissa": 1, "split22": 2, "split211": 3}.get(case, 0)
    S = seed_for(config, case_index)
    prng = random.Random(S + 1)

    if config == 1:
        n = max(1024, int(1_048_576 * scale))
        w = Workload("cfg1_fp32_1Mi_R3", 1, case, 3, 64 * 1024,
                     [TensorSpec("x", (n,), "f32", "normal", 0.02)], S)
        if case != "clean":
            w.patches = [Patch(1, 0, prng.randrange(n), "xor", 1 << prng.randrange(32))]
        return w

    if config == 2:
        n = max(4096, int(25_165_824 * scale))
        w = Workload("cfg2_bf16_bucket_R4", 2, case, 4, 1 << 20,
                     [TensorSpec("bucket", (n,), "bf16", "normal", 1e-3)], S)
        el = prng.randrange(n)
        bit = prng.randrange(7)                       # mantissa bits 0..6
        if case == "mantissa":
            w.patches = [Patch(prng.randrange(4), 0, el, "xor", 1 << bit)]
        elif case == "split22":
            a, b = prng.sample(range(4), 2)
            w.patches = [Patch(a, 0, el, "xor", 1 << bit), Patch(b, 0, el, "xor", 1 << bit)]
        elif case == "split211":
            a, b = prng.sample(range(4), 2)
            per_chunk = w.chunk_bytes // 2
            base = (el // per_chunk) * per_chunk
            span = min(per_chunk, n - base)
            el2 = base + (el - base + 1 + prng.randrange(span - 1)) % span if span > 1 else el
            w.patches = [Patch(a, 0, el, "xor", 1 << bit),
                         Patch(b, 0, el2, "xor", 1 << prng.randrange(7))]
        return w

    if config == 3:
        if scale >= 1.0:
            specs = _cfg3_specs(32, 4096, 14336)
        else:   # keep 7 tensors per layer and the 4:2:1 shape mix, shrink the sizes
            layers = max(1, int(round(32 * min(1.0, scale * 8))))
            d = max(128, int(4096 * math.sqrt(min(1.0, scale * 32 / layers))) // 128 * 128)
            specs = _cfg3_specs(layers, d, d * 7 // 2)
        w = Workload("cfg3_bf16_params_R8", 3, case, 8, 4 << 20, specs, S)
        if case != "clean":
            t_exp, t_nan, t_ulp = prng.sample(range(len(specs)), 3)
            w.patches = [
                Patch(5, t_exp, prng.randrange(specs[t_exp].numel), "xor", 1 << (7 + prng.randrange(8))),
                Patch(5, t_nan, prng.randrange(specs[t_nan].numel), "set", 0x7FC0),
                Patch(5, t_ulp, prng.randrange(specs[t_ulp].numel), "add", prng.choice([1, -1])),
            ]
        return w

    if config == 4:
        n = max(4096, int(1_000_000_000 * scale))
        specs = [TensorSpec("master", (n,), "f32", "normal", 0.02),
                 TensorSpec("exp_avg", (n,), "f32", "normal", 1e-4),
                 TensorSpec("exp_avg_sq", (n,), "f32", "absnormal", 1e-8)]
        w = Workload("cfg4_adam_fp32_R3", 4, case, 3, 16 << 20, specs, S)
        if case != "clean":
            r = prng.randrange(3)
            w.patches = [Patch(r, 2, prng.randrange(n), "xor", 1 << prng.randrange(32))
                         for _ in range(3)]
        return w

    if config == 5:
        n_t = max(8, int(10_000 * scale))
        hi = 4 << 20 if scale >= 1.0 else max(4096, int((4 << 20) * max(scale, 1 / 64)))
        specs = _cfg5_specs(n_t, 256, hi, random.Random(S + 2))
        w = Workload("cfg5_mixed_10k_R16", 5, case, 16, 256 << 10, specs, S)
        if case != "clean":
            ra, rb = prng.sample(range(16), 2)
            ta, tb = prng.sample(range(n_t), 2)
            w.patches = [
                Patch(ra, ta, prng.randrange(specs[ta].numel), "xor",
                      1 << prng.randrange(_int_bits(specs[ta].dtype))),
                Patch(rb, tb, prng.randrange(specs[tb].numel), "xor",
                      1 << prng.randrange(_int_bits(specs[tb].dtype))),
            ]
        return w

    raise ValueError("config must be 1..5")


# ---------------------------------------------------------------- generation

def _fill(view: torch.Tensor, spec: TensorSpec, gen: torch.Generator) -> None:
    if spec.dist == "normal":
        view.normal_(0.0, spec.std, generator=gen)
    elif spec.dist == "absnormal":
        view.normal_(0.0, spec.std, generator=gen)
        view.abs_()
    elif spec.dist == "randint40":
        view.random_(0, 1 << 40, generator=gen)
    elif spec.dist == "randfull":
        view.random_(generator=gen)
    elif spec.dist == "bytes":
        view.random_(0, 256, generator=gen)
    else:
        raise ValueError(spec.dist)


def packed_offsets(specs: Sequence[TensorSpec], align: int = 256) -> Tuple[List[int], int]:
    offs, cur = [], 0
    for s in specs:
        offs.append(cur)
        cur += (s.nbytes + align - 1) // align * align
    return offs, cur


def generate_replica0(w: Workload, device: str = "cpu"):
    """One flat byte buffer holding every tensor at a 256-byte-aligned offset,
    plus the per-tensor typed views into it."""
    offs, total = packed_offsets(w.specs)
    flat = torch.zeros(total, dtype=torch.uint8, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)
    views = tensor_views(flat, w.specs, offs)
    for v, s in zip(views, w.specs):
        _fill(v, s, gen)
    return flat, views


def tensor_views(flat: torch.Tensor, specs: Sequence[TensorSpec], offs=None):
    if offs is None:
        offs, _ = packed_offsets(specs)
    return [flat[o:o + s.nbytes].view(TORCH_DTYPE[s.dtype]) for o, s in zip(offs, specs)]


def generate(w: Workload, device: str = "cpu"):
    """-> (flats, views): R byte buffers and R lists of tensor views, with the
    workload's fault patches already applied."""
    flat0, views0 = generate_replica0(w, device)
    flats, views = [flat0], [views0]
    for _ in range(1, w.R):
        f = flat0.clone()
        flats.append(f)
        views.append(tensor_views(f, w.specs))
    apply_patches(views, w.specs, w.patches)
    return flats, views


def _wrap_signed(value: int, bits: int) -> int:
    value &= (1 << bits) - 1
    return value - (1 << bits) if value >= 1 << (bits - 1) else value


def apply_patches(views, specs: Sequence[TensorSpec], patches: Sequence[Patch]) -> List[int]:
    """Edit element bit patterns in place.  Returns the old patterns (as signed
    integers of the element width) so ``revert_patches`` can undo the edit."""
    old = []
    for p in patches:
        es = DTYPE_BYTES[specs[p.tensor].dtype]
        bits = 8 * es
        iv = views[p.replica][p.tensor].view(-1).view(INT_VIEW[es])
        cur = int(iv[p.element].item())
        old.append(cur)
        if p.op == "xor":
            new = (cur & ((1 << bits) - 1)) ^ (p.value & ((1 << bits) - 1))
        elif p.op == "set":
            new = p.value
        elif p.op == "add":
            new = cur + p.value
        else:
            raise ValueError(p.op)
        iv[p.element] = new if es == 1 else _wrap_signed(new, bits)
    return old


def revert_patches(views, specs: Sequence[TensorSpec], patches: Sequence[Patch],
                   old: Sequence[int]) -> None:
    for p, o in reversed(list(zip(patches, old))):
        es = DTYPE_BYTES[specs[p.tensor].dtype]
        views[p.replica][p.tensor].view(-1).view(INT_VIEW[es])[p.element] = o


def to_numpy_bytes(t: torch.Tensor):
    """Host numpy uint8 view of a tensor's bytes (copies device tensors)."""
    return t.detach().reshape(-1).view(torch.uint8).cpu().numpy()
